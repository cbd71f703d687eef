/*
 * reader_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 CPU statement of what one batched tree-verification
 * step of READER-style lossless speculative decoding computes.  It exists so
 * that the CUDA library can be checked against something that can be read
 * side by side with the paper.  Nothing in the product path may call it, and
 * it shares no code, header, table or helper with the CUDA sources.
 *
 * What each function follows:
 *   oracle_ancestor_matrix  Sec. 3.2 ("Tree Decoding"): the decoding mask M
 *                           with M_ij = 1 iff node i is an ancestor of node j.
 *   oracle_verify_attn      Sec. 3.2: scaled dot-product attention of the
 *                           gamma tree queries against the s cached keys plus
 *                           the gamma tree keys under that mask.
 *   oracle_argmax /         Algorithm 5 (Verify) and Appendix C,
 *   oracle_accept           invariants 1-3 and the deterministic theorem:
 *                           compare the base model's greedy choice with the
 *                           drafted tokens, keep the longest consistent prefix.
 *   oracle_kv_rearrange     Sec. 4.3, Algorithm 4 on the padded batch cache:
 *                           internal padding removed, entries concatenated.
 *   oracle_verify_attn_padded / oracle_padded_append
 *                           Sec. 4.3, the padded batch cache itself: attention under
 *                           its validity mask, and its growth by the batch's longest
 *                           accepted span per step.
 *   oracle_sample_targets   Appendix C, randomized decoding: x* = F(P, U_t) with
 *                           coupled uniforms, temperature inverse-CDF sampling.
 *   oracle_kv_commit        Sec. 4.3 and Algorithm 4 (KVCacheRearrange): the
 *                           accepted entries are concatenated tightly behind
 *                           the committed cache, per sample.
 *
 * Readings taken where the paper is silent (each is listed in the design
 * document as well):
 *   - a node always sees itself (the mask is made reflexive);
 *   - node 0 is the root, parent[0] = -1 and 0 <= parent[j] < j;
 *   - the root is the last committed token: it is always accepted, so the
 *     accepted length counts it and is >= 1;
 *   - argmax ties go to the lowest token id; a NaN never wins a comparison
 *     and a NaN in slot 0 counts as -infinity;
 *   - when several consistent paths have the same length the one ending at
 *     the lowest node index is returned; equal sibling tokens are all
 *     explored;
 *   - nodes deeper than max_path are not candidates (their ancestor at that
 *     depth still is).
 *
 * Pins (tests/test_oracle_*.py, run without a GPU): chain tree == causal
 * attention and single node == decode attention against torch's CPU
 * scaled_dot_product_attention; closed forms (uniform keys -> mean of V, one
 * dominant key -> that V); probabilities sum to one; split-and-merge algebra;
 * sibling-order and page-permutation invariance; exhaustive acceptance on
 * all trees with <= 6 nodes against an independently written accepted-set
 * propagation; Eq. 1 statistics; the deterministic-losslessness loop;
 * random trees and random inputs against torch's attention under a mask
 * derived by transitive closure (to 1e-12).  Every function in this file
 * has at least one pin against something other than itself; none is
 * "parity unpinned".  (The paper prints no worked numeric example, so no
 * pin is a value quoted from it except the Eq. 1 table.)
 *
 * Layouts (row-major, last index fastest):
 *   q, out        [B][T][Hq][D]        k_tree, v_tree  [B][T][Hkv][D]
 *   k_pool,v_pool [num_pages][Hkv][P][D]
 *   page_table    [B][max_pages]       seq_lens [B]    parent [B][T]
 * bf16 values travel as uint16_t bit patterns; widening to double is exact.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum {
    ORACLE_OK = 0,
    ORACLE_BAD_TREE = 2,
    ORACLE_CAPACITY = 3,
    ORACLE_BAD_PAGE = 8
};

static double bf16_bits_to_double(uint16_t bits)
{
    uint32_t u = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Node numbering rule: one root at index 0, every other parent precedes its child. */
int oracle_tree_is_valid(const int32_t *parent, int n_nodes)
{
    if (n_nodes < 1 || parent[0] != -1) return 0;
    for (int j = 1; j < n_nodes; ++j)
        if (parent[j] < 0 || parent[j] >= j) return 0;
    return 1;
}

/* Sec. 3.2: M[i][j] = 1 iff node i is an ancestor of node j (here: or i == j).
 * Found by walking from j towards the root.  M is [T][T], row i, column j. */
void oracle_ancestor_matrix(const int32_t *parent, int n_nodes, uint8_t *M)
{
    memset(M, 0, (size_t)n_nodes * n_nodes);
    for (int j = 0; j < n_nodes; ++j)
        for (int i = j; i >= 0; i = parent[i])
            M[(size_t)i * n_nodes + j] = 1;
}

/* Number of nodes on the path root..j (root has level 1). */
void oracle_levels(const int32_t *parent, int n_nodes, int32_t *level)
{
    for (int j = 0; j < n_nodes; ++j) {
        int c = 0;
        for (int i = j; i >= 0; i = parent[i]) ++c;
        level[j] = c;
    }
}

/*
 * Sec. 3.2 attention.  For sequence b, node j, query head h (KV head h / G):
 * the visible keys are the committed positions 0..L_b-1, reached through the
 * page table, and the tree nodes on the path root..j.  Scores, softmax and
 * the weighted sum of values are all fp64.
 *
 * probs (nullable) receives the softmax weights, [B][T][Hq][probs_stride]:
 * committed position p at column p, tree node i at column L_b + i, zero for
 * keys that are not visible.  lse (nullable) receives log(sum(exp(score))).
 * status[b] != 0 leaves that sequence's outputs at zero.
 */
void oracle_verify_attn(const uint16_t *q, const uint16_t *k_tree, const uint16_t *v_tree,
                        const uint16_t *k_pool, const uint16_t *v_pool,
                        int num_pages, int page_size, int n_kv_heads, int head_dim,
                        const int32_t *page_table, int max_pages, const int32_t *seq_lens,
                        const int32_t *parent, int batch, int n_nodes, int n_q_heads,
                        double scale, double *out, double *lse, double *probs,
                        int64_t probs_stride, int32_t *status)
{
    const int G = n_q_heads / n_kv_heads;
    const int D = head_dim;

    for (int b = 0; b < batch; ++b) {
        int st = ORACLE_OK;
        const int L = seq_lens[b];
        if (!oracle_tree_is_valid(parent + (size_t)b * n_nodes, n_nodes)) st = ORACLE_BAD_TREE;
        else if (L < 0 || (int64_t)L > (int64_t)max_pages * page_size) st = ORACLE_CAPACITY;
        else
            for (int p = 0; p * page_size < L; ++p) {
                int32_t pg = page_table[(size_t)b * max_pages + p];
                if (pg < 0 || pg >= num_pages) st = ORACLE_BAD_PAGE;
            }
        status[b] = st;
    }

    memset(out, 0, sizeof(double) * (size_t)batch * n_nodes * n_q_heads * D);
    if (lse) memset(lse, 0, sizeof(double) * (size_t)batch * n_nodes * n_q_heads);
    if (probs) memset(probs, 0, sizeof(double) * (size_t)batch * n_nodes * n_q_heads * probs_stride);

#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < batch; ++b) {
        for (int h = 0; h < n_q_heads; ++h) {
            if (status[b] != ORACLE_OK) continue;
            const int L = seq_lens[b];
            const int hk = h / G;
            const int32_t *par = parent + (size_t)b * n_nodes;
            double *score = (double *)malloc(sizeof(double) * (size_t)(L + n_nodes));
            const uint16_t **kptr = (const uint16_t **)malloc(sizeof(void *) * (size_t)(L + n_nodes));
            const uint16_t **vptr = (const uint16_t **)malloc(sizeof(void *) * (size_t)(L + n_nodes));
            int64_t *col = (int64_t *)malloc(sizeof(int64_t) * (size_t)(L + n_nodes));

            for (int j = 0; j < n_nodes; ++j) {
                const size_t row = ((size_t)b * n_nodes + j) * n_q_heads + h;
                const uint16_t *qrow = q + row * D;

                /* gather the visible keys */
                int n = 0;
                for (int pos = 0; pos < L; ++pos) {
                    const int32_t pg = page_table[(size_t)b * max_pages + pos / page_size];
                    const size_t at = (((size_t)pg * n_kv_heads + hk) * page_size + pos % page_size) * D;
                    kptr[n] = k_pool + at;
                    vptr[n] = v_pool + at;
                    col[n] = pos;
                    ++n;
                }
                for (int i = j; i >= 0; i = par[i]) {
                    const size_t at = (((size_t)b * n_nodes + i) * n_kv_heads + hk) * D;
                    kptr[n] = k_tree + at;
                    vptr[n] = v_tree + at;
                    col[n] = (int64_t)L + i;
                    ++n;
                }

                /* scores */
                double smax = -INFINITY;
                for (int t = 0; t < n; ++t) {
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d)
                        dot += bf16_bits_to_double(qrow[d]) * bf16_bits_to_double(kptr[t][d]);
                    score[t] = scale * dot;
                    if (score[t] > smax) smax = score[t];
                }
                /* softmax */
                double denom = 0.0;
                for (int t = 0; t < n; ++t) {
                    score[t] = exp(score[t] - smax);
                    denom += score[t];
                }
                /* weighted values */
                double *orow = out + row * D;
                for (int t = 0; t < n; ++t) {
                    const double p = score[t] / denom;
                    if (probs) probs[row * probs_stride + col[t]] = p;
                    for (int d = 0; d < D; ++d)
                        orow[d] += p * bf16_bits_to_double(vptr[t][d]);
                }
                if (lse) lse[row] = smax + log(denom);
            }
            free(score);
            free((void *)kptr);
            free((void *)vptr);
            free(col);
        }
    }
}

/* Greedy policy of Appendix C with a fixed tie-break: first index of the maximum. */
int32_t oracle_argmax_row(const float *row, int64_t vocab)
{
    float best = row[0];
    int64_t at = 0;
    if (isnan(best)) best = -INFINITY;
    for (int64_t v = 1; v < vocab; ++v)
        if (row[v] > best) {
            best = row[v];
            at = v;
        }
    return (int32_t)at;
}

void oracle_argmax(const float *logits, int64_t rows, int64_t vocab, int32_t *target)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        target[r] = oracle_argmax_row(logits + r * vocab, vocab);
}

/*
 * Algorithm 5 (the longest consistent prefix) / Appendix C invariant 2, by brute force: every node e
 * is tried as the end of a root-to-e path; the path is consistent when every
 * non-root node u on it carries the token the base model picks after its
 * parent, tok[u] == target[parent[u]].  The longest consistent path wins,
 * lowest e among equals.  bonus = target[e] is the token invariant 3 commits
 * after the last accepted one.  path is padded with -1.
 */
/*
 * Sec. 4.3 / Algorithm 4 (KVCacheRearrange) on the paper's own layout: a rectangular batch cache
 * k, v [B][Hkv][cap][D] in which every sample's row of `cap` positions holds real entries and
 * internal padding.  valid[b][t] != 0 marks a real entry (a mask, not a test for zero values: a
 * real row may be all zeros).  Per sample: the real entries are moved to the front in their
 * order (RemoveInternalZeroPadding + TightConcatenate), the vacated tail is zeroed, the mask
 * becomes 1...10...0 and lengths[b] is the number of real entries.
 */
void oracle_kv_rearrange(uint16_t *k, uint16_t *v, int B, int Hkv, int cap, int D,
                         uint8_t *valid, int32_t *lengths)
{
    for (int b = 0; b < B; ++b) {
        int n = 0;
        for (int t = 0; t < cap; ++t) {
            if (!valid[(size_t)b * cap + t]) continue;
            for (int h = 0; h < Hkv; ++h) {
                const size_t src = (((size_t)b * Hkv + h) * cap + t) * D;
                const size_t dst = (((size_t)b * Hkv + h) * cap + n) * D;
                if (src != dst) {
                    memmove(k + dst, k + src, (size_t)D * sizeof(uint16_t));
                    memmove(v + dst, v + src, (size_t)D * sizeof(uint16_t));
                }
            }
            ++n;
        }
        for (int h = 0; h < Hkv; ++h) {
            const size_t at = (((size_t)b * Hkv + h) * cap + n) * D;
            memset(k + at, 0, (size_t)(cap - n) * D * sizeof(uint16_t));
            memset(v + at, 0, (size_t)(cap - n) * D * sizeof(uint16_t));
        }
        for (int t = 0; t < cap; ++t) valid[(size_t)b * cap + t] = t < n;
        lengths[b] = n;
    }
}

/*
 * Sec. 4.3, the padded batch cache as the verification attention sees it (the layout the paper
 * starts from, before and between rearrangements): k, v [B][Hkv][cap][D]; every sample's row is
 * used up to the common length *extent; valid[b][t] != 0 marks a real entry, everything else
 * is padding that no query may see.  For sample b, node j, query head h: softmax over the real
 * entries t < extent in position order, then over the tree nodes on root..j (Sec. 3.2).
 * A sample without any real entry attends over its tree path only.
 * status: ORACLE_BAD_TREE per sample; ORACLE_CAPACITY for every sample when extent is outside
 * [0, cap].  Rows of a rejected sample stay zero.
 */
void oracle_verify_attn_padded(const uint16_t *q, const uint16_t *k_tree, const uint16_t *v_tree,
                               const uint16_t *k, const uint16_t *v, int cap, int n_kv_heads, int head_dim,
                               const uint8_t *valid, int extent, const int32_t *parent, int batch,
                               int n_nodes, int n_q_heads, double scale, double *out, double *lse,
                               int32_t *status)
{
    const int G = n_q_heads / n_kv_heads;
    const int D = head_dim;
    memset(out, 0, sizeof(double) * (size_t)batch * n_nodes * n_q_heads * D);
    if (lse) memset(lse, 0, sizeof(double) * (size_t)batch * n_nodes * n_q_heads);
    for (int b = 0; b < batch; ++b) {
        status[b] = ORACLE_OK;
        if (extent < 0 || extent > cap) status[b] = ORACLE_CAPACITY;
        else if (!oracle_tree_is_valid(parent + (size_t)b * n_nodes, n_nodes)) status[b] = ORACLE_BAD_TREE;
    }
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < batch; ++b) {
        for (int h = 0; h < n_q_heads; ++h) {
            if (status[b] != ORACLE_OK) continue;
            const int hk = h / G;
            const int32_t *par = parent + (size_t)b * n_nodes;
            double *score = (double *)malloc(sizeof(double) * (size_t)(extent + n_nodes));
            const uint16_t **kptr = (const uint16_t **)malloc(sizeof(void *) * (size_t)(extent + n_nodes));
            const uint16_t **vptr = (const uint16_t **)malloc(sizeof(void *) * (size_t)(extent + n_nodes));
            for (int j = 0; j < n_nodes; ++j) {
                const size_t row = ((size_t)b * n_nodes + j) * n_q_heads + h;
                const uint16_t *qrow = q + row * D;
                int n = 0;
                for (int t = 0; t < extent; ++t) {
                    if (!valid[(size_t)b * cap + t]) continue;
                    const size_t at = (((size_t)b * n_kv_heads + hk) * cap + t) * D;
                    kptr[n] = k + at;
                    vptr[n] = v + at;
                    ++n;
                }
                for (int i = j; i >= 0; i = par[i]) {
                    const size_t at = (((size_t)b * n_nodes + i) * n_kv_heads + hk) * D;
                    kptr[n] = k_tree + at;
                    vptr[n] = v_tree + at;
                    ++n;
                }
                double smax = -INFINITY;
                for (int t = 0; t < n; ++t) {
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d)
                        dot += bf16_bits_to_double(qrow[d]) * bf16_bits_to_double(kptr[t][d]);
                    score[t] = scale * dot;
                    if (score[t] > smax) smax = score[t];
                }
                double denom = 0.0;
                for (int t = 0; t < n; ++t) {
                    score[t] = exp(score[t] - smax);
                    denom += score[t];
                }
                double *orow = out + row * D;
                for (int t = 0; t < n; ++t) {
                    const double p = score[t] / denom;
                    for (int d = 0; d < D; ++d)
                        orow[d] += p * bf16_bits_to_double(vptr[t][d]);
                }
                if (lse) lse[row] = smax + log(denom);
            }
            free(score);
            free((void *)kptr);
            free((void *)vptr);
        }
    }
}

/*
 * Sec. 4.3, how the padded batch cache grows in one step: the accepted span of sample b (the K/V
 * rows of path[b][0 .. n_acc[b]-1]) is written at positions extent .. extent + n_acc[b] - 1 of its
 * row and marked real; the row is then filled with zero rows, marked padding, up to the batch's
 * new common length extent + max_b n_acc[b] ("other prompts are padded with zeros to match the new
 * maximum length").  *extent becomes that length.
 * All or nothing: when the new length exceeds cap, or some n_acc is outside [0, max_path], or a
 * path entry is not a node, every status is ORACLE_CAPACITY and nothing is changed.
 */
void oracle_padded_append(uint16_t *k, uint16_t *v, int B, int Hkv, int cap, int D, uint8_t *valid,
                          int32_t *extent, const uint16_t *k_tree, const uint16_t *v_tree, int n_nodes,
                          const int32_t *path, const int32_t *n_acc, int max_path, int32_t *status)
{
    const int E = *extent;
    int grow = 0, ok = E >= 0 && E <= cap;
    for (int b = 0; b < B; ++b) {
        if (n_acc[b] < 0 || n_acc[b] > max_path) { ok = 0; continue; }
        if (n_acc[b] > grow) grow = n_acc[b];
        for (int i = 0; i < n_acc[b]; ++i) {
            const int32_t node = path[(size_t)b * max_path + i];
            if (node < 0 || node >= n_nodes) ok = 0;
        }
    }
    if (ok && (int64_t)E + grow > cap) ok = 0;
    for (int b = 0; b < B; ++b) status[b] = ok ? ORACLE_OK : ORACLE_CAPACITY;
    if (!ok) return;
    for (int b = 0; b < B; ++b) {
        for (int i = 0; i < grow; ++i) {
            const int t = E + i;
            const int real = i < n_acc[b];
            valid[(size_t)b * cap + t] = (uint8_t)real;
            for (int h = 0; h < Hkv; ++h) {
                const size_t dst = (((size_t)b * Hkv + h) * cap + t) * D;
                if (real) {
                    const size_t src = (((size_t)b * n_nodes + path[(size_t)b * max_path + i]) * Hkv + h) * D;
                    memcpy(k + dst, k_tree + src, sizeof(uint16_t) * D);
                    memcpy(v + dst, v_tree + src, sizeof(uint16_t) * D);
                } else {
                    memset(k + dst, 0, sizeof(uint16_t) * D);
                    memset(v + dst, 0, sizeof(uint16_t) * D);
                }
            }
        }
    }
    *extent = E + grow;
}

/*
 * Randomized policy of Appendix C ("Randomized decoding"): x* = F(P_theta(. | prefix), U_t), one
 * uniform U_t per output POSITION, shared by the base run and the verifier.  Every node at tree
 * level lv (root = 1) proposes a token for position lv, and its target is the token the policy emits
 * for position lv + 1: all nodes of one level therefore use the same uniform, u[b][lv - 1].
 *
 * F is temperature sampling by inverse CDF, stated so that a float never decides the token by a
 * rounding that depends on summation order:
 *   c    = (float)(log2(e) / temperature)                 (double division, rounded once)
 *   m    = row maximum (NaN never wins; NaN in slot 0 counts as -inf)
 *   x_v  = (l_v - m) * c          two fp32 operations; NaN or x_v < -64 gives weight 0
 *   n    = nearest integer to x_v (ties to even), f = x_v - n in [-1/2, 1/2]
 *   p    = 1 + f(c1 + f(c2 + f(c3 + f(c4 + f c5))))      fp32 Horner with fused multiply-adds,
 *          c_k = ln(2)^k / k! rounded to fp32            (2^f to about 3e-6)
 *   W_v  = trunc(p * 2^(n + 40))                          integer weight, at most 2^40
 *   S    = sum_v W_v (exact, 64-bit);  U = trunc(u * 2^24);  thr = (S * U) >> 24 (exact, 128-bit)
 *   x*   = the first v whose inclusive prefix sum of W exceeds thr      (0 if S = 0)
 * Top-k filtering (top_k >= 1; 0 = off): tau = the top_k-th largest logit of the row (NaN counts as
 * -inf); only logits >= tau keep their weight, so logits equal to tau are all kept (the usual
 * "mask what is below the k-th value" rule) and the kept set can exceed top_k on ties.
 * Top-p filtering (0 < top_p < 1; >= 1 = off), applied to what top-k left: with S0 the sum of the kept
 * weights and M = max(1, (S0 * trunc(top_p * 2^24)) >> 24), tau_p is the largest logit value t for
 * which the weights of all kept logits >= t add up to at least M (the smallest nucleus reaching
 * top_p, with logits equal to the last admitted value all admitted); only logits >= tau_p stay.
 * Ties on "measure-zero boundaries" are thus resolved towards the lower token id.
 */
static uint64_t sample_weight(float l, float m, float c)
{
    const float x = (l - m) * c;
    if (!(x >= -64.0f)) return 0;                 /* also catches NaN */
    const float n = nearbyintf(x);                /* default rounding mode: ties to even */
    const float f = x - n;
    float p = 1.3333558146e-3f;
    p = fmaf(p, f, 9.6181291076e-3f);
    p = fmaf(p, f, 5.5504108665e-2f);
    p = fmaf(p, f, 2.4022650696e-1f);
    p = fmaf(p, f, 6.9314718056e-1f);
    p = fmaf(p, f, 1.0f);
    return (uint64_t)ldexpf(p, (int)n + 40);      /* exact scaling, then truncation */
}

typedef struct { float l; uint64_t w; } logit_weight;

static int cmp_lw_desc(const void *a, const void *b)
{
    const float x = ((const logit_weight *)a)->l, y = ((const logit_weight *)b)->l;
    return (x < y) - (x > y);
}

static int cmp_float_desc(const void *a, const void *b)
{
    const float x = *(const float *)a, y = *(const float *)b;
    return (x < y) - (x > y);
}

int32_t oracle_sample_row(const float *row, int64_t vocab, float u, double temperature, int64_t top_k, float top_p)
{
    const float c = (float)(1.4426950408889634 / temperature);
    float m = row[0];
    if (isnan(m)) m = -INFINITY;
    for (int64_t v = 1; v < vocab; ++v)
        if (row[v] > m) m = row[v];
    if (m == -INFINITY) return 0;                 /* nothing has weight */
    float tau = -INFINITY;                        /* the top_k-th largest logit */
    if (top_k > 0 && top_k < vocab) {
        float *tmp = (float *)malloc((size_t)vocab * sizeof(float));
        for (int64_t v = 0; v < vocab; ++v) tmp[v] = isnan(row[v]) ? -INFINITY : row[v];
        qsort(tmp, (size_t)vocab, sizeof(float), cmp_float_desc);
        tau = tmp[top_k - 1];
        free(tmp);
    }
    uint64_t total = 0;
    for (int64_t v = 0; v < vocab; ++v) total += row[v] >= tau ? sample_weight(row[v], m, c) : 0;
    if (total == 0) return 0;
    if (top_p < 1.0f) {                           /* the nucleus among what top-k left */
        if (!(top_p >= 5.9604645e-8f)) top_p = 5.9604645e-8f;      /* 2^-24; also NaN */
        uint64_t need = (uint64_t)(((unsigned __int128)total * (uint64_t)(top_p * 16777216.0f)) >> 24);
        if (need == 0) need = 1;
        logit_weight *lw = (logit_weight *)malloc((size_t)vocab * sizeof(logit_weight));
        int64_t n = 0;
        for (int64_t v = 0; v < vocab; ++v)
            if (row[v] >= tau) { lw[n].l = row[v]; lw[n].w = sample_weight(row[v], m, c); ++n; }
        qsort(lw, (size_t)n, sizeof(logit_weight), cmp_lw_desc);
        uint64_t cum = 0;
        for (int64_t i = 0; i < n;) {             /* one group of equal logits at a time */
            int64_t j = i;
            while (j < n && lw[j].l == lw[i].l) cum += lw[j++].w;
            if (cum >= need) { tau = lw[i].l; break; }
            i = j;
        }
        free(lw);
        total = cum;                              /* the weights of the logits >= the new tau */
    }
    if (!(u >= 0.0f)) u = 0.0f;                              /* u is meant to lie in [0, 1) */
    if (u > 0.99999994f) u = 0.99999994f;
    const uint64_t U = (uint64_t)(u * 16777216.0f);          /* 24 bits */
    const uint64_t thr = (uint64_t)(((unsigned __int128)total * U) >> 24);
    uint64_t run = 0;
    for (int64_t v = 0; v < vocab; ++v) {
        run += row[v] >= tau ? sample_weight(row[v], m, c) : 0;
        if (run > thr) return (int32_t)v;
    }
    return (int32_t)(vocab - 1);                  /* not reached: thr < total */
}

/* target[b][j] for every node; uniforms f32 [B][T], entry lv - 1 serves the nodes of level lv. */
void oracle_sample_targets(const float *logits, const int32_t *parent, const float *uniforms,
                           int B, int T, int64_t vocab, double temperature, int64_t top_k, float top_p,
                           int32_t *target)
{
    /* One uniform per output position (Appendix C): position = tree level, taken from
     * oracle_levels, the same function the attention pins use.  Only for a parent
     * array that is not a tree (no level exists) is a position made up, by counting
     * the nodes met while the parent index keeps decreasing, so that any input gives
     * a defined result. */
    int32_t *level = (int32_t *)malloc(sizeof(int32_t) * (size_t)B * T);
    if (!level) return;
    for (int b = 0; b < B; ++b) {
        const int32_t *par = parent + (size_t)b * T;
        if (oracle_tree_is_valid(par, T)) {
            oracle_levels(par, T, level + (size_t)b * T);
            continue;
        }
        for (int j = 0; j < T; ++j) {
            int count = 0;
            for (int i = j, steps = 0; i >= 0 && i < T && steps < T; ++steps) {
                ++count;
                i = par[i] < i ? par[i] : -1;
            }
            level[(size_t)b * T + j] = count;
        }
    }
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < (int64_t)B * T; ++r) {
        const int b = (int)(r / T);
        target[r] = oracle_sample_row(logits + r * vocab, vocab, uniforms[(size_t)b * T + level[r] - 1], temperature, top_k, top_p);
    }
    free(level);
}

void oracle_accept(const int32_t *parent, const int32_t *tok, const int32_t *target,
                   int batch, int n_nodes, int max_path,
                   int32_t *path, int32_t *n_acc, int32_t *bonus, int32_t *status)
{
    for (int b = 0; b < batch; ++b) {
        const int32_t *par = parent + (size_t)b * n_nodes;
        const int32_t *tk = tok + (size_t)b * n_nodes;
        const int32_t *tg = target + (size_t)b * n_nodes;
        int32_t *pth = path + (size_t)b * max_path;
        for (int k = 0; k < max_path; ++k) pth[k] = -1;
        n_acc[b] = 0;
        bonus[b] = -1;
        if (!oracle_tree_is_valid(par, n_nodes)) {
            status[b] = ORACLE_BAD_TREE;
            continue;
        }
        status[b] = ORACLE_OK;
        int best_len = 0, best_end = -1;
        for (int e = 0; e < n_nodes; ++e) {
            int len = 0, ok = 1;
            for (int u = e; u >= 0; u = par[u]) {
                ++len;
                if (par[u] >= 0 && tk[u] != tg[par[u]]) ok = 0;
            }
            if (ok && len <= max_path && len > best_len) {
                best_len = len;
                best_end = e;
            }
        }
        if (best_end < 0) continue; /* only when max_path < 1 */
        n_acc[b] = best_len;
        bonus[b] = tg[best_end];
        int k = best_len - 1;
        for (int u = best_end; u >= 0; u = par[u]) pth[k--] = u;
    }
}

/*
 * Sec. 4.3 / Algorithm 4 in per-step form: the K/V rows of the accepted nodes
 * are appended, in path order and without gaps, at logical positions
 * L_b .. L_b + n_acc - 1 of sequence b; the physical slot of position p is
 * page_table[b][p / P] * P + p % P.  A sequence whose pages cannot hold the
 * new positions, or that would write below the shared prefix, gets
 * ORACLE_CAPACITY and is left untouched.  slots is padded with -1.
 */
void oracle_kv_commit(uint16_t *k_pool, uint16_t *v_pool, int num_pages, int page_size,
                      int n_kv_heads, int head_dim, const int32_t *page_table, int max_pages,
                      int32_t *seq_lens, int shared_prefix_len,
                      const uint16_t *k_tree, const uint16_t *v_tree, int batch, int n_nodes,
                      const int32_t *path, const int32_t *n_acc, int max_path,
                      int update_seq_lens, int32_t *slots, int32_t *status)
{
    const int D = head_dim;
    for (int b = 0; b < batch; ++b) {
        int32_t *sl = slots + (size_t)b * max_path;
        for (int k = 0; k < max_path; ++k) sl[k] = -1;
        const int L = seq_lens[b];
        const int n = n_acc[b];
        status[b] = ORACLE_OK;
        if (n <= 0) continue;
        int ok = (n <= max_path) && L >= 0 && L >= shared_prefix_len &&
                 ((int64_t)L + n <= (int64_t)max_pages * page_size);
        for (int k = 0; ok && k < n; ++k) {
            const int32_t pg = page_table[(size_t)b * max_pages + (L + k) / page_size];
            const int32_t node = path[(size_t)b * max_path + k];
            if (pg < 0 || pg >= num_pages || node < 0 || node >= n_nodes) ok = 0;
        }
        if (!ok) {
            status[b] = ORACLE_CAPACITY;
            continue;
        }
        for (int k = 0; k < n; ++k) {
            const int pos = L + k;
            const int32_t pg = page_table[(size_t)b * max_pages + pos / page_size];
            const int32_t node = path[(size_t)b * max_path + k];
            sl[k] = pg * page_size + pos % page_size;
            for (int h = 0; h < n_kv_heads; ++h) {
                const size_t dst = (((size_t)pg * n_kv_heads + h) * page_size + pos % page_size) * D;
                const size_t src = (((size_t)b * n_nodes + node) * n_kv_heads + h) * D;
                memcpy(k_pool + dst, k_tree + src, sizeof(uint16_t) * D);
                memcpy(v_pool + dst, v_tree + src, sizeof(uint16_t) * D);
            }
        }
        if (update_seq_lens) seq_lens[b] = L + n;
    }
}
