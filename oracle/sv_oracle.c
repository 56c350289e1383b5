/*
 * sv_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of the importance-based sparse
 * verification attention of the paper "Accelerate Speculative Decoding with
 * Sparse Computation in Verification" (Section 3.1 "Sparse Attention",
 * Section 3.2 "Piecewise Budget Control", Section 3.3 "Inter-layer Retrieval
 * Reuse").  Only the tests, the smoke check and the CPU-baseline leg of the
 * benchmark may call it.  It shares no code with the CUDA library and is
 * written so that each function can be checked against the paper by eye:
 * no blocking, no fusion, no reordering beyond what the definitions state.
 *
 * Every floating-point quantity is fp64.  Tensor inputs arrive as bfloat16
 * bit patterns (uint16) and are widened exactly.
 *
 * KV-cache layout (Eq. 4: one block = one KV head x B consecutive tokens):
 *   pool[page][h][t_in_block][d], page = block_table[s][t / B].
 *
 * Parity pins (see tests/test_oracle_pins.py):
 *   svo_block_reps / svo_group_query / svo_scores : Eq. 5 evaluated literally
 *       in numpy; planted-shift closed form.
 *   svo_select  : brute-force enumeration of all subsets on tiny inputs.
 *   svo_verify_attn : budget = all blocks equals svo_dense_verify_attn and a
 *       library scaled-dot-product attention with an explicit mask; prefix
 *       truncation; softmax weights sum to one; log-sum-exp split merge.
 *   svo_budget_blocks : closed form of Eq. 6 and the sparsity column of Table 2.
 *   svo_kv_append : the appended cache read back with numpy indexing equals old tokens followed by the
 *       accepted rows; one call equals token-by-token calls; attention afterwards equals attention on a
 *       cache built with the longer prefix.
 *   svo_jaccard_adjacent / svo_pick_anchors : Python set arithmetic on random subsets; identical layers give
 *       J = 1, disjoint ones 0; numpy argsort for the top-K.
 *   svo_group_query_row / svo_select_global / svo_pair_overlap (retrieval variants the paper discusses):
 *       row 0 equals svo_group_query; brute-force enumeration over all (head, block) subsets on tiny inputs,
 *       one KV head equals svo_select, numpy lexsort; Python set intersections.
 *   svo_accept (Eq. 2-3): identical models accept everything and sample from the target (numpy searchsorted);
 *       a one-hot target reduces to greedy prefix matching; the emitted token is distributed as the target,
 *       summed exactly over the draft token(s) for one draft token and for two siblings.
 *   Approximation quality of sparse vs dense attention: parity unpinned (the
 *       paper bounds nothing; reported as information only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_f64(uint16_t bits)
{
    uint32_t u = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int svo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* element d of the cached key/value of token t, kv head h, sequence s */
static double kv_at(const uint16_t *pool, const int32_t *block_table, int s, int h, int64_t t, int d,
                    int Hkv, int D, int B, int NBmax)
{
    int64_t page = block_table[(int64_t)s * NBmax + t / B];
    int64_t off = ((page * Hkv + h) * B + (t % B)) * D + d;
    return bf16_to_f64(pool[off]);
}

/*
 * Block representative (Eq. 5 by linearity: s = q0 . mean(k)): the mean key of
 * the block.  The last block of a sequence may hold fewer than B tokens; its
 * mean is taken over the tokens it holds.
 * reps[s][h][b][d], b < ceil(L_s / B); other entries are left untouched.
 */
int svo_block_reps(int S, int Hkv, int D, int B, int NBmax, const uint16_t *k_pool, const int32_t *block_table,
                   const int32_t *seq_lens, double *reps)
{
    for (int s = 0; s < S; ++s) {
        int64_t L = seq_lens[s];
        int nb = (int)((L + B - 1) / B);
        if (nb > NBmax) return 1;
#pragma omp parallel for collapse(2)
        for (int h = 0; h < Hkv; ++h) {
            for (int b = 0; b < nb; ++b) {
                int64_t t0 = (int64_t)b * B;
                int64_t cnt = (L - t0 < B) ? (L - t0) : B;
                for (int d = 0; d < D; ++d) {
                    double sum = 0.0;
                    for (int64_t t = t0; t < t0 + cnt; ++t)
                        sum += kv_at(k_pool, block_table, s, h, t, d, Hkv, D, B, NBmax);
                    reps[(((int64_t)s * Hkv + h) * NBmax + b) * D + d] = sum / (double)cnt;
                }
            }
        }
    }
    return 0;
}

/*
 * Retrieval query (Section 2.2: only the first draft token retrieves).  Blocks
 * belong to KV heads, queries to query heads; the G = Hq / Hkv query heads
 * hq = h*G .. h*G+G-1 share KV head h, and the retrieval query of KV head h is
 * their mean.  q[s][i][hq][d], row i = 0 is the first draft token.
 * qbar[s][h][d].
 */
int svo_group_query(int S, int T, int Hq, int Hkv, int D, const uint16_t *q, double *qbar)
{
    if (Hq % Hkv) return 1;
    int G = Hq / Hkv;
    for (int s = 0; s < S; ++s)
        for (int h = 0; h < Hkv; ++h)
            for (int d = 0; d < D; ++d) {
                double sum = 0.0;
                for (int g = 0; g < G; ++g)
                    sum += bf16_to_f64(q[(((int64_t)s * T + 0) * Hq + h * G + g) * D + d]);
                qbar[((int64_t)s * Hkv + h) * D + d] = sum / (double)G;
            }
    return 0;
}

/* Importance score (Eq. 5): scores[s][h][b] = qbar[s][h] . reps[s][h][b].  No 1/sqrt(D), no softmax. */
int svo_scores(int S, int Hkv, int D, int B, int NBmax, const double *qbar, const double *reps,
               const int32_t *seq_lens, double *scores)
{
    for (int s = 0; s < S; ++s) {
        int nb = (int)(((int64_t)seq_lens[s] + B - 1) / B);
        for (int h = 0; h < Hkv; ++h)
            for (int b = 0; b < nb; ++b) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d)
                    acc += qbar[((int64_t)s * Hkv + h) * D + d] * reps[(((int64_t)s * Hkv + h) * NBmax + b) * D + d];
                scores[((int64_t)s * Hkv + h) * NBmax + b] = acc;
            }
    }
    return 0;
}

/*
 * Block selection (Section 3.1): keep the first n_sink and the last n_local
 * blocks without eviction, then the highest-scoring blocks of the rest until
 * budget[s] blocks are kept (the forced blocks count against the budget).
 * Equal scores: the smaller block index wins.  A budget >= the number of
 * blocks keeps every block (Section 3.2: no eviction).  One set per
 * (sequence, KV head), shared by every draft token (Section 2.2).
 * idx[s][h][0..cnt) ascending block indices, cnt[s][h].
 * Returns 2 when the forced blocks alone exceed the budget, 3 when the set
 * does not fit max_sel.
 */
int svo_select(int S, int Hkv, int B, int NBmax, const double *scores, const int32_t *seq_lens,
               const int32_t *budget, int n_sink, int n_local, int max_sel, int32_t *idx, int32_t *cnt)
{
    for (int s = 0; s < S; ++s) {
        int nb = (int)(((int64_t)seq_lens[s] + B - 1) / B);
        int N = budget[s];
        for (int h = 0; h < Hkv; ++h) {
            const double *sc = scores + ((int64_t)s * Hkv + h) * NBmax;
            int32_t *out = idx + ((int64_t)s * Hkv + h) * max_sel;
            char *keep = (char *)calloc((size_t)(nb > 0 ? nb : 1), 1);
            int kept = 0;
            if (N >= nb) {
                for (int b = 0; b < nb; ++b) keep[b] = 1;
                kept = nb;
            } else {
                for (int b = 0; b < nb; ++b)
                    if (b < n_sink || b >= nb - n_local) {
                        keep[b] = 1;
                        ++kept;
                    }
                if (kept > N) {
                    free(keep);
                    return 2;
                }
                while (kept < N) {
                    int best = -1;
                    for (int b = 0; b < nb; ++b)
                        if (!keep[b] && (best < 0 || sc[b] > sc[best])) best = b;
                    keep[best] = 1;
                    ++kept;
                }
            }
            if (kept > max_sel) {
                free(keep);
                return 3;
            }
            int n = 0;
            for (int b = 0; b < nb; ++b)
                if (keep[b]) out[n++] = b;
            cnt[(int64_t)s * Hkv + h] = n;
            free(keep);
        }
    }
    return 0;
}

/* is draft token j visible to draft token i?  chain: j <= i; tree: j is i or an ancestor of i. */
static int draft_visible(const int32_t *parent, int s, int T, int i, int j)
{
    if (!parent) return j <= i;
    for (int a = i; a >= 0; a = parent[(int64_t)s * T + a])
        if (a == j) return 1;
    return 0;
}

/*
 * softmax(scale * q . k) weighted sum of v over a list of (z, value-row) pairs,
 * the textbook three steps: max, exponentials, normalised sum.
 */
static void softmax_weighted_sum(int n, const double *z, const double *vals, int D, double *o, double *lse)
{
    double m = -INFINITY, l = 0.0;
    for (int j = 0; j < n; ++j)
        if (z[j] > m) m = z[j];
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    for (int j = 0; j < n; ++j) {
        double p = exp(z[j] - m);
        l += p;
        for (int d = 0; d < D; ++d) o[d] += p * vals[(int64_t)j * D + d];
    }
    for (int d = 0; d < D; ++d) o[d] /= l;
    *lse = m + log(l);
}

/*
 * Sparse verification attention (Fig. 1; the 4B(1-s_a)T^2 d term of Table 1):
 * every draft token i of every query head hq attends to the cached tokens of
 * the selected blocks of its KV head hq / G (tokens t < L_s only) and to the
 * draft tokens visible to it (itself and its ancestors; a causal chain when
 * parent is NULL).  Standard scaled dot-product attention.
 *
 * samples: NULL -> all (s, i, hq) rows; otherwise n_samples triples
 * (s, i, hq) and out/lse hold n_samples rows in that order.
 * out[s][i][hq][d] fp64, lse[s][i][hq] = log of the softmax denominator.
 */
int svo_verify_attn(int S, int T, int Hq, int Hkv, int D, int B, int NBmax, const uint16_t *q,
                    const uint16_t *k_pool, const uint16_t *v_pool, const int32_t *block_table,
                    const int32_t *seq_lens, const uint16_t *draft_k, const uint16_t *draft_v,
                    const int32_t *parent, const int32_t *sel_idx, const int32_t *sel_cnt, int max_sel,
                    double scale, int n_samples, const int32_t *samples, double *out, double *lse)
{
    int G = Hq / Hkv;
    int64_t n_rows = samples ? n_samples : (int64_t)S * T * Hq;
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        int s, i, hq;
        if (samples) {
            s = samples[3 * r], i = samples[3 * r + 1], hq = samples[3 * r + 2];
        } else {
            s = (int)(r / ((int64_t)T * Hq)), i = (int)((r / Hq) % T), hq = (int)(r % Hq);
        }
        int h = hq / G;
        int64_t L = seq_lens[s];
        const int32_t *sel = sel_idx + ((int64_t)s * Hkv + h) * max_sel;
        int n_sel = sel_cnt[(int64_t)s * Hkv + h];
        int64_t cap = (int64_t)n_sel * B + T;
        double *z = (double *)malloc(sizeof(double) * (size_t)cap);
        double *vals = (double *)malloc(sizeof(double) * (size_t)cap * D);
        double qi[1024];
        if (!z || !vals || D > 1024) {
            err = 1;
            free(z);
            free(vals);
            continue;
        }
        for (int d = 0; d < D; ++d) qi[d] = bf16_to_f64(q[(((int64_t)s * T + i) * Hq + hq) * D + d]);
        int n = 0;
        for (int j = 0; j < n_sel; ++j) {
            int64_t b = sel[j];
            for (int64_t t = b * B; t < (b + 1) * B && t < L; ++t) {
                double dot = 0.0;
                for (int d = 0; d < D; ++d) dot += qi[d] * kv_at(k_pool, block_table, s, h, t, d, Hkv, D, B, NBmax);
                z[n] = scale * dot;
                for (int d = 0; d < D; ++d)
                    vals[(int64_t)n * D + d] = kv_at(v_pool, block_table, s, h, t, d, Hkv, D, B, NBmax);
                ++n;
            }
        }
        for (int j = 0; j < T; ++j) {
            if (!draft_visible(parent, s, T, i, j)) continue;
            const uint16_t *kj = draft_k + (((int64_t)s * T + j) * Hkv + h) * D;
            const uint16_t *vj = draft_v + (((int64_t)s * T + j) * Hkv + h) * D;
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += qi[d] * bf16_to_f64(kj[d]);
            z[n] = scale * dot;
            for (int d = 0; d < D; ++d) vals[(int64_t)n * D + d] = bf16_to_f64(vj[d]);
            ++n;
        }
        softmax_weighted_sum(n, z, vals, D, out + r * D, lse + r);
        free(z);
        free(vals);
    }
    return err;
}

/*
 * Dense ("strict") verification attention: the same attention over the whole
 * cached prefix 0..L_s-1, written as its own contiguous loop with no block
 * list.  Fixed point of the sparse path when nothing is evicted, and the dense
 * CPU baseline.  Same sampling convention as svo_verify_attn.
 */
int svo_dense_verify_attn(int S, int T, int Hq, int Hkv, int D, int B, int NBmax, const uint16_t *q,
                          const uint16_t *k_pool, const uint16_t *v_pool, const int32_t *block_table,
                          const int32_t *seq_lens, const uint16_t *draft_k, const uint16_t *draft_v,
                          const int32_t *parent, double scale, int n_samples, const int32_t *samples,
                          double *out, double *lse)
{
    int G = Hq / Hkv;
    int64_t n_rows = samples ? n_samples : (int64_t)S * T * Hq;
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        int s, i, hq;
        if (samples) {
            s = samples[3 * r], i = samples[3 * r + 1], hq = samples[3 * r + 2];
        } else {
            s = (int)(r / ((int64_t)T * Hq)), i = (int)((r / Hq) % T), hq = (int)(r % Hq);
        }
        int h = hq / G;
        int64_t L = seq_lens[s];
        int64_t n = L + T;
        double *z = (double *)malloc(sizeof(double) * (size_t)n);
        if (!z) {
            err = 1;
            continue;
        }
        const uint16_t *qi = q + (((int64_t)s * T + i) * Hq + hq) * D;
        for (int64_t t = 0; t < L; ++t) {
            double dot = 0.0;
            for (int d = 0; d < D; ++d)
                dot += bf16_to_f64(qi[d]) * kv_at(k_pool, block_table, s, h, t, d, Hkv, D, B, NBmax);
            z[t] = scale * dot;
        }
        for (int j = 0; j < T; ++j) {
            if (!draft_visible(parent, s, T, i, j)) {
                z[L + j] = -INFINITY;
                continue;
            }
            const uint16_t *kj = draft_k + (((int64_t)s * T + j) * Hkv + h) * D;
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += bf16_to_f64(qi[d]) * bf16_to_f64(kj[d]);
            z[L + j] = scale * dot;
        }
        double m = -INFINITY;
        for (int64_t t = 0; t < n; ++t)
            if (z[t] > m) m = z[t];
        double l = 0.0;
        for (int64_t t = 0; t < n; ++t) {
            z[t] = exp(z[t] - m); /* z now holds the unnormalised softmax weights */
            l += z[t];
        }
        double *o = out + r * D;
        for (int d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int64_t t = 0; t < L; ++t)
                acc += z[t] / l * kv_at(v_pool, block_table, s, h, t, d, Hkv, D, B, NBmax);
            for (int j = 0; j < T; ++j)
                acc += z[L + j] / l * bf16_to_f64(draft_v[(((int64_t)s * T + j) * Hkv + h) * D + d]);
            o[d] = acc;
        }
        lse[r] = m + log(l);
        free(z);
    }
    return err;
}

/*
 * Piecewise budget (Section 3.2, Eq. 6) per KV head: a cache of at most L0
 * tokens is not evicted; a longer one keeps ((L - L0) * rho + L0) / B blocks
 * per head, rounded up, and never fewer than the forced blocks nor more than
 * the blocks that exist.
 */
int svo_budget_blocks(int64_t L, int64_t L0, double rho, int B, int n_sink, int n_local)
{
    int nb = (int)((L + B - 1) / B);
    if (L <= L0) return nb;
    double tokens = ((double)(L - L0)) * rho + (double)L0;
    int n = (int)ceil(tokens / (double)B);
    int forced = n_sink + n_local;
    if (n < forced) n = forced;
    if (n > nb) n = nb;
    return n;
}

/*
 * Commit of accepted draft tokens (Section 2.1: the accepted prefix of the draft is kept, the rest
 * discarded; Section 3.1: blocks are cut from the *current* KV cache).  For every sequence the K/V rows of
 * the accepted draft tokens accept_idx[s][0 .. n_accept[s]) are appended, in that order, at positions
 * L_s, L_s + 1, ... of the paged cache (the pages must already be in block_table), the length grows by
 * n_accept[s], and the representatives of the blocks that received tokens are recomputed as in
 * svo_block_reps.  Pools are modified in place; new lengths go to seq_lens_out.
 */
int svo_kv_append(int S, int T, int Hkv, int D, int B, int NBmax, uint16_t *k_pool, uint16_t *v_pool,
                  const int32_t *block_table, const int32_t *seq_lens, const uint16_t *draft_k,
                  const uint16_t *draft_v, const int32_t *accept_idx, const int32_t *n_accept, int max_accept,
                  int32_t *seq_lens_out, double *reps)
{
    for (int s = 0; s < S; ++s) {
        int64_t L = seq_lens[s];
        int n = n_accept[s];
        if (n < 0 || n > max_accept || (L + n + B - 1) / B > NBmax) return 1;
        for (int a = 0; a < n; ++a) {
            int j = accept_idx[(int64_t)s * max_accept + a];
            if (j < 0 || j >= T) return 2;
            int64_t t = L + a;
            int64_t page = block_table[(int64_t)s * NBmax + t / B];
            for (int h = 0; h < Hkv; ++h)
                for (int d = 0; d < D; ++d) {
                    int64_t dst = ((page * Hkv + h) * B + (t % B)) * D + d;
                    int64_t src = (((int64_t)s * T + j) * Hkv + h) * D + d;
                    k_pool[dst] = draft_k[src];
                    v_pool[dst] = draft_v[src];
                }
        }
        int64_t Ln = L + n;
        seq_lens_out[s] = (int32_t)Ln;
        if (n == 0 || !reps) continue;
        for (int64_t b = L / B; b <= (Ln - 1) / B; ++b) {
            int64_t t0 = b * B;
            int64_t cnt = (Ln - t0 < B) ? (Ln - t0) : B;
            for (int h = 0; h < Hkv; ++h)
                for (int d = 0; d < D; ++d) {
                    double sum = 0.0;
                    for (int64_t t = t0; t < t0 + cnt; ++t)
                        sum += kv_at(k_pool, block_table, s, h, t, d, Hkv, D, B, NBmax);
                    reps[(((int64_t)s * Hkv + h) * NBmax + b) * D + d] = sum / (double)cnt;
                }
        }
    }
    return 0;
}

/*
 * Anchor-layer calibration (Section 3.3, Eq. 7-8).  Input: the block sets kept by every layer for a batch
 * of calibration samples (idx[l][s][h][0..cnt[l][s][h])).  The mask M_l of a sample spans all its
 * candidate blocks (every KV head); adjacent layers are compared by the Jaccard similarity
 * J(M_l, M_{l-1}) = |M_l n M_{l-1}| / |M_l u M_{l-1}| (Eq. 7), averaged over the samples, with
 * J(M_1, M_0) = 0 for the first layer by definition.  inter/uni[l][s] are the set sizes, J[l] the mean.
 */
int svo_jaccard_adjacent(int n_layers, int S, int Hkv, int max_sel, const int32_t *idx, const int32_t *cnt,
                         int32_t *inter, int32_t *uni, double *J)
{
    for (int l = 0; l < n_layers; ++l) {
        double sum = 0.0;
        for (int s = 0; s < S; ++s) {
            int in = 0, un = 0;
            if (l > 0) {
                for (int h = 0; h < Hkv; ++h) {
                    const int32_t *a = idx + ((((int64_t)l * S + s) * Hkv + h) * max_sel);
                    const int32_t *b = idx + ((((int64_t)(l - 1) * S + s) * Hkv + h) * max_sel);
                    int na = cnt[((int64_t)l * S + s) * Hkv + h], nb = cnt[((int64_t)(l - 1) * S + s) * Hkv + h];
                    int common = 0;
                    for (int i = 0; i < na; ++i)
                        for (int j = 0; j < nb; ++j)
                            if (a[i] == b[j]) ++common;
                    in += common;
                    un += na + nb - common;
                }
                sum += un > 0 ? (double)in / (double)un : 1.0;   /* two empty masks are identical */
            }
            inter[(int64_t)l * S + s] = in;
            uni[(int64_t)l * S + s] = un;
        }
        J[l] = l > 0 ? sum / (double)S : 0.0;
    }
    return 0;
}

/*
 * Eq. 8: the K layers with the lowest similarity to their predecessor (largest 1 - J) become anchors;
 * equal similarities: the earlier layer first.  anchors[l] = 1 / 0.
 */
int svo_pick_anchors(int n_layers, const double *J, int K, uint8_t *anchors)
{
    if (K < 1 || K > n_layers) return 1;
    for (int l = 0; l < n_layers; ++l) anchors[l] = 0;
    for (int k = 0; k < K; ++k) {
        int best = -1;
        for (int l = 0; l < n_layers; ++l)
            if (!anchors[l] && (best < 0 || 1.0 - J[l] > 1.0 - J[best])) best = l;
        anchors[best] = 1;
    }
    return 0;
}

/*
 * Retrieval variants the paper discusses but does not adopt.
 *
 * (1) Retrieval query of draft token `row` (Section 2.2 measures how much the blocks retrieved by different
 *     draft tokens "based on their respective query values" overlap): the group mean of that token's query
 *     heads.  row = 0 is svo_group_query.
 */
int svo_group_query_row(int S, int T, int Hq, int Hkv, int D, const uint16_t *q, int row, double *qbar)
{
    if (Hq % Hkv || row < 0 || row >= T) return 1;
    int G = Hq / Hkv;
    for (int s = 0; s < S; ++s)
        for (int h = 0; h < Hkv; ++h)
            for (int d = 0; d < D; ++d) {
                double sum = 0.0;
                for (int g = 0; g < G; ++g)
                    sum += bf16_to_f64(q[(((int64_t)s * T + row) * Hq + h * G + g) * D + d]);
                qbar[((int64_t)s * Hkv + h) * D + d] = sum / (double)G;
            }
    return 0;
}

/*
 * (2) Budget shared by the KV heads (Eq. 6 counts N_budget = ... x H / B blocks over all heads): the
 *     budget[s] * Hkv best (head, block) pairs of a sequence are kept, whichever head they belong to.
 *     The first n_sink and last n_local blocks of every head are kept first and count against the total.
 *     Equal scores: the smaller head, then the smaller block index wins.  budget[s] >= number of blocks
 *     keeps everything.  idx[s][h][0..cnt[s][h]) ascending.  Returns 2 when the forced blocks exceed the
 *     total, 3 when a head's set does not fit max_sel.
 */
int svo_select_global(int S, int Hkv, int B, int NBmax, const double *scores, const int32_t *seq_lens,
                      const int32_t *budget, int n_sink, int n_local, int max_sel, int32_t *idx, int32_t *cnt)
{
    for (int s = 0; s < S; ++s) {
        int nb = (int)(((int64_t)seq_lens[s] + B - 1) / B);
        int64_t total = (int64_t)budget[s] * Hkv;
        char *keep = (char *)calloc((size_t)(nb > 0 ? (int64_t)nb * Hkv : 1), 1);
        int64_t kept = 0;
        if (budget[s] >= nb) {
            for (int64_t e = 0; e < (int64_t)nb * Hkv; ++e) keep[e] = 1;
        } else {
            for (int h = 0; h < Hkv; ++h)
                for (int b = 0; b < nb; ++b)
                    if (b < n_sink || b >= nb - n_local) {
                        keep[(int64_t)h * nb + b] = 1;
                        ++kept;
                    }
            if (kept > total) {
                free(keep);
                return 2;
            }
            while (kept < total) {
                int bh = -1, bb = -1;
                for (int h = 0; h < Hkv; ++h)
                    for (int b = 0; b < nb; ++b) {
                        if (keep[(int64_t)h * nb + b]) continue;
                        double v = scores[((int64_t)s * Hkv + h) * NBmax + b];
                        if (bh < 0 || v > scores[((int64_t)s * Hkv + bh) * NBmax + bb]) bh = h, bb = b;
                    }
                keep[(int64_t)bh * nb + bb] = 1;
                ++kept;
            }
        }
        for (int h = 0; h < Hkv; ++h) {
            int n = 0;
            for (int b = 0; b < nb; ++b)
                if (keep[(int64_t)h * nb + b]) {
                    if (n >= max_sel) {
                        free(keep);
                        return 3;
                    }
                    idx[((int64_t)s * Hkv + h) * max_sel + n++] = b;
                }
            cnt[(int64_t)s * Hkv + h] = n;
        }
        free(keep);
    }
    return 0;
}

/*
 * (3) Overlap of the blocks retrieved by two draft tokens (Section 2.2, the block-overlap figure): the size
 *     of the intersection of their sets, per (sequence, KV head).  idx[i][s][h][0..cnt[i][s][h]) is the set
 *     of draft token i.  inter[s][h][i][j] = |Sel_i n Sel_j| (the diagonal is the set size).
 */
int svo_pair_overlap(int T, int S, int Hkv, int max_sel, const int32_t *idx, const int32_t *cnt, int32_t *inter)
{
    for (int s = 0; s < S; ++s)
        for (int h = 0; h < Hkv; ++h)
            for (int i = 0; i < T; ++i)
                for (int j = 0; j < T; ++j) {
                    const int32_t *a = idx + (((int64_t)i * S + s) * Hkv + h) * max_sel;
                    const int32_t *b = idx + (((int64_t)j * S + s) * Hkv + h) * max_sel;
                    int na = cnt[((int64_t)i * S + s) * Hkv + h], nb = cnt[((int64_t)j * S + s) * Hkv + h];
                    int common = 0;
                    for (int x = 0; x < na; ++x)
                        for (int y = 0; y < nb; ++y)
                            if (a[x] == b[y]) ++common;
                    inter[((((int64_t)s * Hkv + h) * T) + i) * T + j] = common;
                }
    return 0;
}

/*
 * Acceptance of the draft tokens after verification (Section 2.1, Eq. 2-3).
 *
 * Rows of a step: row 0 is the token accepted in the previous step (the root), rows 1..T-1 the draft tokens;
 * parent[s][i] < i is the row a draft token continues (NULL: the chain parent[i] = i - 1).  p_target[s][i][:]
 * is the target model's distribution of the token that follows row i, p_draft[s][i][:] the draft model's
 * distribution the children of row i were drawn from (fp32 probabilities, widened exactly).
 *
 * Walk from the root.  At row `cur` with current target distribution p (initially p_target[cur]) and draft
 * distribution q = p_draft[cur], the children of cur are tried in row order: child c with token x is accepted
 * with probability alpha = min(1, p(x) / q(x)) (Eq. 2), i.e. when u_accept[s][c] < alpha; the walk moves to c.
 * A rejected child replaces p by norm(max(0, p - q)) (Eq. 3) before the next sibling is tried (a chain has no
 * sibling: that case is Eq. 2-3 verbatim; for several siblings drawn independently from q this is the
 * multi-round rule that keeps the output distributed as the target).  When no child is accepted (or cur is a
 * leaf) the next token is drawn from the current p -- the adjusted distribution after a rejection, the
 * target's own distribution after a fully accepted path -- by inversion of its cumulative sum in vocabulary
 * order with u_next[s]: the smallest x with sum_{y<=x} p(y) >= u_next * sum_y p(y).  Everything after the
 * first rejection on the path is discarded.
 *
 * A residual that is zero everywhere (p == q) leaves p unchanged.  q(x) = 0 gives alpha = 1.
 *
 * Outputs: path[s][0..n_path[s]) = rows whose tokens are kept (root first, then the accepted drafts in
 * order); next_token[s]; alpha[s][c] for every child that was tried (NaN otherwise); final_dist[s][:]
 * (optional) the normalised distribution next_token was drawn from.
 */
int svo_accept(int S, int T, int V, const float *p_target, const float *p_draft, const int32_t *tokens,
               const int32_t *parent, const float *u_accept, const float *u_next, int32_t *path, int32_t *n_path,
               int32_t *next_token, double *alpha, double *final_dist)
{
    double *p = (double *)malloc(sizeof(double) * (size_t)V);
    if (!p) return 1;
    for (int s = 0; s < S; ++s) {
        const int32_t *tok = tokens + (int64_t)s * T;
        for (int i = 0; i < T; ++i) alpha[(int64_t)s * T + i] = NAN;
        int cur = 0, n = 0;
        path[(int64_t)s * T + n++] = 0;
        for (;;) {
            const float *pt = p_target + ((int64_t)s * T + cur) * V;
            const float *q = p_draft + ((int64_t)s * T + cur) * V;
            for (int x = 0; x < V; ++x) p[x] = (double)pt[x];
            int moved = 0;
            for (int c = cur + 1; c < T; ++c) {
                int par = parent ? parent[(int64_t)s * T + c] : c - 1;
                if (par != cur) continue;
                int x = tok[c];
                if (x < 0 || x >= V) {
                    free(p);
                    return 2;
                }
                double qx = (double)q[x];
                double a = (qx <= 0.0 || p[x] >= qx) ? 1.0 : p[x] / qx;
                alpha[(int64_t)s * T + c] = a;
                if ((double)u_accept[(int64_t)s * T + c] < a) {
                    path[(int64_t)s * T + n++] = c;
                    cur = c;
                    moved = 1;
                    break;
                }
                /* rejected: p <- norm(max(0, p - q)) (Eq. 3) */
                double z = 0.0;
                for (int y = 0; y < V; ++y) {
                    double d = p[y] - (double)q[y];
                    z += d > 0.0 ? d : 0.0;
                }
                if (z > 0.0)
                    for (int y = 0; y < V; ++y) {
                        double d = p[y] - (double)q[y];
                        p[y] = d > 0.0 ? d / z : 0.0;
                    }
            }
            if (moved) continue;
            double tot = 0.0;
            for (int y = 0; y < V; ++y) tot += p[y];
            double target = (double)u_next[s] * tot, run = 0.0;
            int pick = V - 1;
            for (int y = 0; y < V; ++y) {
                run += p[y];
                if (run >= target && p[y] > 0.0) {
                    pick = y;
                    break;
                }
            }
            next_token[s] = pick;
            if (final_dist)
                for (int y = 0; y < V; ++y) final_dist[(int64_t)s * V + y] = tot > 0.0 ? p[y] / tot : 0.0;
            break;
        }
        n_path[s] = n;
        for (int i = n; i < T; ++i) path[(int64_t)s * T + i] = -1;
    }
    free(p);
    return 0;
}

/*
 * Representatives stored in bfloat16 (storage variant of Eq. 5's block representative): the fp64 mean is
 * rounded once, to the nearest bfloat16 (8 significand bits), ties to even; scores are then taken with the
 * rounded values.  Magnitudes here are far from the bfloat16 range limits; subnormal results are not handled
 * specially (frexp/ldexp keep them exact anyway).
 */
int svo_round_bf16(int64_t n, const double *x, double *y)
{
    for (int64_t i = 0; i < n; ++i) {
        double v = x[i];
        if (v == 0.0 || !isfinite(v)) {
            y[i] = v;
            continue;
        }
        int e;
        double m = frexp(v, &e);          /* v = m * 2^e, 0.5 <= |m| < 1 */
        double scaled = ldexp(m, 8);      /* 8 significand bits: |scaled| in [128, 256) */
        double r = nearbyint(scaled);     /* default rounding mode: to nearest, ties to even */
        y[i] = ldexp(r, e - 8);
    }
    return 0;
}
