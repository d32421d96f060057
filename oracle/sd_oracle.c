/*
 * Reference checker for draft-tree verification (TEST INFRASTRUCTURE ONLY).
 *
 * Plain, slow, fp64 CPU statement of what the target model's batched
 * verification of a draft token tree computes.  The paper (Hyper-Bagel,
 * Sec. 1 and Sec. 3.1) says only that the draft's speculative tokens are
 * validated by the target model in one parallel pass and (Sec. 4.1) that the
 * target's outputs are unchanged by it; because the result is exactly that of
 * greedy decoding, every function below is the plain definition written out:
 *
 *   orc_attention  softmax attention of every tree node over the cached prefix
 *                  plus its own ancestors in the tree
 *   orc_lmhead     logits = hidden . W^T, lowest-index argmax, top-2 values
 *   orc_accept     deepest node whose whole root path matches the target
 *   orc_compact    accepted tree rows copied behind the prefix in the cache
 *
 * Inputs are bf16 bit patterns (uint16) widened exactly to double.  No
 * blocking, fusion or reordering beyond the definitions.  Nothing here is
 * shared with, or used by, the GPU library; only tests, the smoke check and
 * the CPU-baseline leg of the benchmark call it.
 *
 * Numeric agreement with the paper's reported acceptance lengths and
 * tokens/s is "parity unpinned": those need trained models and data.
 * Every function here is pinned by closed forms, brute force and library
 * cross-checks in the CPU test-suite.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_to_double(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* geometry shared by the calls; all arrays are host memory */
typedef struct {
    int32_t B, T_max, Hq, Hkv, D, block, max_blocks;
    const int32_t *block_table; /* [B][max_blocks]            */
    const int32_t *len;         /* [B] cached prefix lengths  */
    const int32_t *n_nodes;     /* [B]                        */
    const int32_t *parents;     /* [B][T_max], parents[b][0] = -1 */
} orc_geom;

/* element offset of (logical token t, kv head) of sequence b in a paged cache
 * laid out [block][Hkv][block_size][D] */
static inline size_t cache_row(const orc_geom *g, int b, int t, int kvh)
{
    int blk = g->block_table[(size_t)b * g->max_blocks + t / g->block];
    return (((size_t)blk * g->Hkv + kvh) * g->block + (t % g->block)) * (size_t)g->D;
}

/*
 * One output row of tree attention (Sec. 1: the target validates all
 * speculative tokens in one pass; Sec. 4.1: results equal the target's own).
 * Query (b, node i, head h) sees every cached prefix key t < len[b] and the
 * tree keys of node i and of all its ancestors; nothing else enters the sums.
 */
static void attention_row(const orc_geom *g, const uint16_t *kc, const uint16_t *vc,
                          const uint16_t *q, const uint16_t *kt, const uint16_t *vt,
                          double scale, int b, int i, int h, double *out, double *lse)
{
    const int D = g->D;
    const int G = g->Hq / g->Hkv;
    const int kvh = h / G;
    const int P = g->len[b];
    const uint16_t *qr = q + (((size_t)b * g->T_max + i) * g->Hq + h) * D;

    /* visible tree nodes: i, parent(i), ..., root */
    int anc[64];
    int na = 0;
    for (int j = i; j >= 0; j = g->parents[(size_t)b * g->T_max + j])
        anc[na++] = j;

    const int nkeys = P + na;
    double *s = (double *)malloc(sizeof(double) * (size_t)nkeys);
    double m = -INFINITY;
    for (int t = 0; t < nkeys; ++t) {
        const uint16_t *kr = (t < P)
            ? kc + cache_row(g, b, t, kvh)
            : kt + (((size_t)b * g->T_max + anc[t - P]) * g->Hkv + kvh) * D;
        double acc = 0.0;
        for (int d = 0; d < D; ++d)
            acc += bf16_to_double(qr[d]) * bf16_to_double(kr[d]);
        s[t] = acc * scale;
        if (s[t] > m) m = s[t];
    }
    double denom = 0.0;
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    for (int t = 0; t < nkeys; ++t) {
        const uint16_t *vr = (t < P)
            ? vc + cache_row(g, b, t, kvh)
            : vt + (((size_t)b * g->T_max + anc[t - P]) * g->Hkv + kvh) * D;
        double w = exp(s[t] - m);
        denom += w;
        for (int d = 0; d < D; ++d)
            out[d] += w * bf16_to_double(vr[d]);
    }
    for (int d = 0; d < D; ++d) out[d] /= denom;
    if (lse) *lse = m + log(denom);
    free(s);
}

/* all rows: out [B][T_max][Hq][D] double, lse [B][T_max][Hq] double
 * (rows of nodes >= n_nodes[b] are left untouched) */
void orc_attention(const orc_geom *g, const uint16_t *kc, const uint16_t *vc,
                   const uint16_t *q, const uint16_t *kt, const uint16_t *vt,
                   double scale, double *out, double *lse)
{
    const long rows = (long)g->B * g->T_max * g->Hq;
#pragma omp parallel for schedule(dynamic, 4)
    for (long r = 0; r < rows; ++r) {
        int h = (int)(r % g->Hq);
        int i = (int)((r / g->Hq) % g->T_max);
        int b = (int)(r / ((long)g->Hq * g->T_max));
        if (i >= g->n_nodes[b]) continue;
        attention_row(g, kc, vc, q, kt, vt, scale, b, i, h,
                      out + (size_t)r * g->D, lse ? lse + r : NULL);
    }
}

/* sampled rows: triples (b,i,h) in rows[3*n]; out [n][D], lse [n] */
void orc_attention_rows(const orc_geom *g, const uint16_t *kc, const uint16_t *vc,
                        const uint16_t *q, const uint16_t *kt, const uint16_t *vt,
                        double scale, const int32_t *rows, int n, double *out, double *lse)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n; ++r)
        attention_row(g, kc, vc, q, kt, vt, scale, rows[3 * r], rows[3 * r + 1], rows[3 * r + 2],
                      out + (size_t)r * g->D, lse ? lse + r : NULL);
}

/*
 * LM head: logits[r][v] = sum_k hidden[r][k] * W[v][k]; for every requested
 * row the lowest index attaining the maximum, the maximum and the runner-up
 * value (the target's greedy token at each tree node, Sec. 1 / Sec. 4.1).
 * rows == NULL means all M rows; otherwise n_rows row indices.
 */
void orc_lmhead(const uint16_t *hidden, const uint16_t *W, int M, int Hd, int V,
                const int32_t *rows, int n_rows,
                int32_t *argmax, double *top1, double *top2)
{
    const int n = rows ? n_rows : M;
    double *hd = (double *)malloc(sizeof(double) * (size_t)n * Hd);
    for (int r = 0; r < n; ++r) {
        int src = rows ? rows[r] : r;
        for (int k = 0; k < Hd; ++k)
            hd[(size_t)r * Hd + k] = bf16_to_double(hidden[(size_t)src * Hd + k]);
        argmax[r] = -1;
        top1[r] = -INFINITY;
        top2[r] = -INFINITY;
    }
    /* vocabulary entries are visited in increasing order inside every thread's
     * contiguous slab, so "strictly greater" keeps the lowest index */
#pragma omp parallel
    {
        double *wv = (double *)malloc(sizeof(double) * (size_t)Hd);
        int32_t *la = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
        double *l1 = (double *)malloc(sizeof(double) * (size_t)n);
        double *l2 = (double *)malloc(sizeof(double) * (size_t)n);
        for (int r = 0; r < n; ++r) { la[r] = -1; l1[r] = -INFINITY; l2[r] = -INFINITY; }
#pragma omp for schedule(static)
        for (int v = 0; v < V; ++v) {
            for (int k = 0; k < Hd; ++k) wv[k] = bf16_to_double(W[(size_t)v * Hd + k]);
            for (int r = 0; r < n; ++r) {
                const double *hr = hd + (size_t)r * Hd;
                double acc = 0.0;
#pragma omp simd reduction(+ : acc)
                for (int k = 0; k < Hd; ++k) acc += hr[k] * wv[k];
                if (acc > l1[r]) { l2[r] = l1[r]; l1[r] = acc; la[r] = v; }
                else if (acc > l2[r]) { l2[r] = acc; }
            }
        }
#pragma omp critical
        {
            for (int r = 0; r < n; ++r) {
                if (la[r] < 0) continue;
                /* merge (l1,l2,la) of this slab into the global result */
                if (l1[r] > top1[r] || (l1[r] == top1[r] && la[r] < argmax[r])) {
                    double old1 = top1[r];
                    top1[r] = l1[r];
                    argmax[r] = la[r];
                    double c = old1 > l2[r] ? old1 : l2[r];
                    if (c > top2[r]) top2[r] = c;
                } else {
                    if (l1[r] > top2[r]) top2[r] = l1[r];
                }
            }
        }
        free(wv); free(la); free(l1); free(l2);
    }
    free(hd);
}

/* full logits for small cases: logits [M][V] double */
void orc_logits(const uint16_t *hidden, const uint16_t *W, int M, int Hd, int V, double *logits)
{
#pragma omp parallel for schedule(static)
    for (int v = 0; v < V; ++v)
        for (int r = 0; r < M; ++r) {
            double acc = 0.0;
            for (int k = 0; k < Hd; ++k)
                acc += bf16_to_double(hidden[(size_t)r * Hd + k]) * bf16_to_double(W[(size_t)v * Hd + k]);
            logits[(size_t)r * V + v] = acc;
        }
}

/*
 * Greedy acceptance (Sec. 1 "validated"; Sec. 4.1: lossless, and the reported
 * statistic is the average acceptance length).  A non-root node j matches when
 * its draft token equals the target's token at its parent.  A node is valid
 * when every non-root node on its root path matches.  The answer is the valid
 * node of greatest depth, the smallest index among equals.
 *   n_acc   = depth + 1 (the root is always accepted)
 *   path    = root ... node
 *   out_tok = draft tokens of path[1..] followed by the target's token at the
 *             last accepted node (the bonus token): n_acc tokens
 *   new_len = len + n_acc
 * Entries of path/out_tok beyond n_acc are set to -1.
 * Returns 0, or -2 when a parent array is not a tree with parent < child.
 */
int orc_accept(const orc_geom *g, const int32_t *draft_tok, const int32_t *target,
               int32_t *n_acc, int32_t *path, int32_t *out_tok, int32_t *new_len)
{
    const int T = g->T_max;
    for (int b = 0; b < g->B; ++b) {
        const int32_t *par = g->parents + (size_t)b * T;
        const int32_t *dt = draft_tok + (size_t)b * T;
        const int32_t *tg = target + (size_t)b * T;
        const int n = g->n_nodes[b];
        if (n < 1 || n > T || par[0] != -1) return -2;
        for (int i = 1; i < n; ++i)
            if (par[i] < 0 || par[i] >= i) return -2;
        int best = 0, best_depth = 0;
        for (int i = 0; i < n; ++i) {
            int ok = 1, depth = 0;
            for (int j = i; j > 0; j = par[j]) {
                if (dt[j] != tg[par[j]]) ok = 0;
                ++depth;
            }
            if (ok && depth > best_depth) { best = i; best_depth = depth; }
        }
        const int na = best_depth + 1;
        n_acc[b] = na;
        for (int k = 0; k < T; ++k) { path[(size_t)b * T + k] = -1; out_tok[(size_t)b * T + k] = -1; }
        int j = best;
        for (int k = na - 1; k >= 0; --k) { path[(size_t)b * T + k] = j; j = par[j]; }
        for (int k = 1; k < na; ++k) out_tok[(size_t)b * T + k - 1] = dt[path[(size_t)b * T + k]];
        out_tok[(size_t)b * T + na - 1] = tg[best];
        new_len[b] = g->len[b] + na;
    }
    return 0;
}

/*
 * Compaction of accepted KV (Sec. 4.1 describes the KV cache as the running
 * context): for k < n_acc[b], cache slot len[b]+k of sequence b receives tree
 * row path[b][k], every KV head, K and V, verbatim.  One layer per call.
 */
void orc_compact(const orc_geom *g, uint16_t *kc, uint16_t *vc,
                 const uint16_t *kt, const uint16_t *vt,
                 const int32_t *n_acc, const int32_t *path)
{
    const int D = g->D;
    for (int b = 0; b < g->B; ++b)
        for (int k = 0; k < n_acc[b]; ++k) {
            int node = path[(size_t)b * g->T_max + k];
            for (int kvh = 0; kvh < g->Hkv; ++kvh) {
                size_t dst = cache_row(g, b, g->len[b] + k, kvh);
                size_t src = (((size_t)b * g->T_max + node) * g->Hkv + kvh) * D;
                memcpy(kc + dst, kt + src, sizeof(uint16_t) * (size_t)D);
                memcpy(vc + dst, vt + src, sizeof(uint16_t) * (size_t)D);
            }
        }
}
