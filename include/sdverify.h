/*
 * sdverify — batched verification of a draft token tree on one B200.
 *
 * Hyper-Bagel (arXiv 2509.18824) accelerates next-token prediction by
 * speculative decoding: a light draft model proposes several tokens and the
 * target model validates all of them in one parallel pass (Sec. 1), which
 * trades the memory-access bottleneck of autoregressive decoding for a
 * computational one; the target's outputs are unchanged (Sec. 4.1).  This
 * library is that validation pass, split into its four data-parallel parts:
 *
 *   sd_verify_attention  attention of every tree node over the cached prefix
 *                        KV and over its own ancestors' KV (per layer)
 *   sd_lmhead_argmax     target's greedy token at every tree node
 *   sd_accept_tree       longest root path whose drafts the target confirms
 *   sd_compact_kv        accepted nodes' KV appended to the cache (all layers)
 *
 * Conventions common to every call
 *   - "dev" pointers are device memory on the current CUDA device, "host"
 *     pointers are ordinary host memory.  The caller owns every buffer; the
 *     library allocates nothing and frees nothing.
 *   - bf16 tensors are passed as void* / uint16 bit patterns.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and
 *     return without synchronising.
 *   - Host-detectable problems (null or misaligned pointers, unsupported
 *     shapes, workspace too small) return a negative sd_status before anything
 *     is launched.  Problems only visible on the device (bad parent array,
 *     block-table entry out of range, an expired bounded wait) store the first
 *     error code into *dev_status (int32, dev, must be 0 on entry) and the
 *     kernel finishes normally; outputs are unspecified in that case.
 *   - Same inputs give bit-identical outputs from run to run.
 *   - All dev pointers must be 16-byte aligned.
 *
 * Layouts
 *   KV cache of one layer, K and V each:  bf16 [num_blocks][Hkv][64][D]
 *       (block = 64 tokens; one (block, head) tile is 16 KiB contiguous)
 *   logical token t of sequence b lives in block block_table[b][t / 64],
 *       slot t % 64.  Slots at or beyond len[b], and the tree K/V rows of nodes at or
 *       beyond n_nodes[b], may hold any bit pattern (NaN and infinity included): they never reach a sum.
 *   q, out:            bf16 [B][T_max][Hq][D]
 *   tree K, tree V:    bf16 [B][T_max][Hkv][D]
 *   query head h uses KV head h / (Hq / Hkv).
 *   Node 0 of a tree is the root (the last emitted token, whose KV is not yet
 *   cached); parents[b][0] = -1 and 0 <= parents[b][i] < i.
 *
 * Supported: D = 128, block_size = 64, 1 <= T_max <= 64, Hq % Hkv == 0,
 * Hq / Hkv <= 8.
 */
#ifndef SDVERIFY_H
#define SDVERIFY_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SD_OK = 0,
    SD_ERR_INVALID_ARG = -1,
    SD_ERR_INVALID_TREE = -2,
    SD_ERR_UNSUPPORTED = -3,
    SD_ERR_WORKSPACE = -4,
    SD_ERR_CUDA = -5,
    SD_ERR_TIMEOUT = -6,
    SD_ERR_BOUNDS = -7
} sd_status;

/* Paged KV cache of ONE layer (dev memory owned by the caller). */
typedef struct {
    void *k;             /* dev bf16 [num_blocks][Hkv][64][D] */
    void *v;             /* dev bf16 [num_blocks][Hkv][64][D] */
    int32_t num_blocks;
} sd_kv_layer;

/* Batch geometry shared by the calls.  Scalars are host values; pointers are
 * dev arrays owned by the caller. */
typedef struct {
    int32_t B;                   /* sequences                                        */
    int32_t T_max;               /* row stride of per-node arrays; 1..64             */
    int32_t Hq, Hkv, D;          /* query heads, KV heads, head dim (128)            */
    int32_t block_size;          /* 64                                               */
    int32_t max_blocks_per_seq;  /* row stride of block_table                        */
    const int32_t *block_table;  /* dev [B][max_blocks_per_seq]; covers len+n_nodes  */
    const int32_t *len;          /* dev [B] cached prefix length of each sequence    */
    const int32_t *n_nodes;      /* dev [B] nodes in each tree, 1..T_max             */
    const int32_t *parents;      /* dev [B][T_max]                                   */
    uint64_t *anc_mask;          /* dev [B][T_max]; bit j of [b][i] set iff node j is
                                    i itself or an ancestor of i (sd_tree_prepare)   */
} sd_batch;

/* Library version (major*100 + minor). */
int sd_version(void);

/* Static, human-readable name of a status code. */
const char *sd_status_string(sd_status s);

/*
 * Scratch bytes that sd_verify_attention (for this geometry; only the host
 * scalars of *geom are read) and sd_lmhead_argmax / sd_lmhead_accept_compact
 * (for M rows, vocabulary V) need; the larger of the two.  Pass M = 0 or V = 0 to size for attention
 * only, geom = NULL for the LM head only.
 */
size_t sd_workspace_bytes(const sd_batch *geom, int32_t M, int32_t V);

/*
 * Ancestor masks of the draft trees (Sec. 1: the speculative tokens are
 * validated together; a node may attend only to its own root path).
 * Validates parents (root -1, parent < child, n_nodes in 1..T_max) and fills
 * batch->anc_mask.  A bad tree stores SD_ERR_INVALID_TREE into *dev_status.
 */
sd_status sd_tree_prepare(const sd_batch *batch, int32_t *dev_status, void *stream);

/*
 * Tree-masked GQA attention of one layer (Sec. 1, batched validation; Sec. 4.1,
 * results equal the target's own decoding).  For sequence b, node i < n_nodes[b]
 * and query head h:  out = softmax(scale * q . K^T) V  over the keys
 * { cached tokens t < len[b] } U { tree nodes j with bit j set in anc_mask[b][i] }.
 *   q, k_tree, v_tree : dev bf16, layouts above (read only)
 *   out               : dev bf16 [B][T_max][Hq][D]; rows of nodes >= n_nodes[b] are zeroed
 *   lse               : dev f32 [B][T_max][Hq] or NULL; natural-log sum of exp of the scaled scores
 *   workspace         : dev scratch of at least sd_workspace_bytes(batch, 0, 0)
 * Arithmetic: bf16 inputs, fp32 accumulation, bf16 output (round to nearest even).
 * Needs batch->anc_mask filled.  Errors: SD_ERR_INVALID_ARG, SD_ERR_UNSUPPORTED,
 * SD_ERR_WORKSPACE (workspace_bytes below sd_workspace_bytes) on the host;
 * SD_ERR_BOUNDS (block-table entry outside [0, num_blocks), or len[b] needs
 * more than max_blocks_per_seq blocks) or SD_ERR_TIMEOUT through *dev_status.
 */
sd_status sd_verify_attention(const sd_batch *batch, const sd_kv_layer *cache,
                              const void *q, const void *k_tree, const void *v_tree,
                              float scale, void *out, float *lse,
                              void *workspace, size_t workspace_bytes,
                              int32_t *dev_status, void *stream);

/*
 * The same attention for L layers in one call (Sec. 1: one parallel validation
 * pass of the target model; every layer attends over its own cache and its own
 * tree K/V with the same trees and masks).  Layer l computes exactly what
 * sd_verify_attention computes from caches[l], q_layers[l], k_tree_layers[l],
 * v_tree_layers[l] into out_layers[l] (and lse_layers[l]), to within fp32
 * rounding (the keys of a sequence may be split into a different number of
 * chunks than in a single-layer call).  The layers are independent, so they
 * share kernel launches: the grid runs over (layer, sequence, KV head, row
 * tile), which fills the GPU without splitting the keys of a sequence and
 * hides every per-launch cost but one.  Usable when all layers' q and tree K/V
 * exist before the call (as in this library's verify step, where they are
 * inputs); a decoder that produces them layer by layer calls
 * sd_verify_attention per layer instead.
 *   caches                     : host array [L] of cache descriptors
 *   q_layers, k_tree_layers,
 *   v_tree_layers, out_layers  : host arrays [L] of dev pointers, layouts above
 *   lse_layers                 : NULL, or host array [L] of dev pointers (entries may be NULL)
 * The host arrays are read before the call returns.  Errors as sd_verify_attention.
 */
sd_status sd_verify_attention_layers(const sd_batch *batch, const sd_kv_layer *caches, int32_t L,
                                     const void *const *q_layers, const void *const *k_tree_layers,
                                     const void *const *v_tree_layers, float scale,
                                     void *const *out_layers, float *const *lse_layers,
                                     void *workspace, size_t workspace_bytes,
                                     int32_t *dev_status, void *stream);

/*
 * LM-head projection with fused arg-max (Sec. 1 / Sec. 4.1: the target's own
 * greedy prediction at every speculative position).
 *   logits[r][v] = sum_k hidden[r][k] * W[v][k]     (never written to memory)
 *   argmax[r]    = lowest v attaining max_v logits[r][v]
 *   maxlogit[r]  = that maximum (fp32), optional
 *   hidden : dev bf16 [M][Hd]      W : dev bf16 [V][Hd]  (row-major, Hd contiguous)
 *   Hd % 64 == 0, V >= 1, M >= 1
 *   workspace : dev scratch of at least sd_workspace_bytes(NULL, M, V)
 * Arithmetic: bf16 products accumulated in fp32.
 */
sd_status sd_lmhead_argmax(const void *hidden, const void *W,
                           int32_t M, int32_t Hd, int32_t V,
                           int32_t *argmax, float *maxlogit,
                           void *workspace, size_t workspace_bytes,
                           int32_t *dev_status, void *stream);

/*
 * sd_lmhead_argmax without any scratch argument.  (The paper has no counterpart
 * to this call; it exists for the way some programs have to use the library.)
 *
 * Who needs it: code that is not allowed to obtain device memory at the point
 * where it verifies a draft - a decode loop whose memory was budgeted and
 * carved up once at start-up, a plug-in running inside a server that hands it
 * a fixed arena, a latency-critical path where cudaMalloc's implicit device
 * synchronisation is unacceptable.  Such callers cannot size and allocate the
 * workspace sd_lmhead_argmax asks for, so here the library brings its own: a
 * fixed 1 MiB table compiled into the library image, resident on every GPU
 * that loads the library until the process ends.  This call allocates and
 * frees nothing, on the host or on the device.
 *
 * Same arithmetic, arguments and results as sd_lmhead_argmax, with these
 * differences:
 *   - M is limited to SD_LMHEAD_STATIC_MAX_ROWS (512) rows per call, the
 *     number the built-in table holds; larger M returns SD_ERR_UNSUPPORTED and
 *     launches nothing (call it once per slice of rows instead).
 *   - The first call on each device looks up the table's device address.
 *     Make that first call during start-up, before any stream capture begins,
 *     and from one host thread (later calls may come from any thread).
 *   - All calls on a device share the one table, and it keeps whatever the
 *     previous call left in it.  No entry needs clearing between calls (each
 *     call overwrites every entry it later reads), but two calls whose kernels
 *     overlap on the GPU - different streams, no ordering between them - race
 *     on it and give wrong answers.  Keep calls on one stream, or order them.
 */
#define SD_LMHEAD_STATIC_MAX_ROWS 512
sd_status sd_lmhead_argmax_static(const void *hidden, const void *W,
                                  int32_t M, int32_t Hd, int32_t V,
                                  int32_t *argmax, float *maxlogit,
                                  int32_t *dev_status, void *stream);

/*
 * Greedy acceptance (Sec. 1 "validated"; Sec. 4.1 reports the average
 * acceptance length this step produces).  Node j >= 1 matches when
 * draft_tok[b][j] == target_argmax[b][parents[b][j]]; a node is valid when
 * every non-root node on its root path matches; the valid node of greatest
 * depth wins, the smallest index among equals.
 *   n_acc[b]    = its depth + 1 (the root always counts)
 *   path[b][k]  = k-th node from the root, k < n_acc[b]; -1 beyond
 *   out_tok[b]  = draft tokens of path[b][1..], then target_argmax at the last
 *                 accepted node (bonus token): n_acc[b] tokens; -1 beyond
 *   new_len[b]  = len[b] + n_acc[b]
 * All arrays dev int32: draft_tok, target_argmax, path, out_tok [B][T_max];
 * n_acc, new_len [B].  A bad parent array stores SD_ERR_INVALID_TREE.
 */
sd_status sd_accept_tree(const sd_batch *batch, const int32_t *draft_tok,
                         const int32_t *target_argmax,
                         int32_t *n_acc, int32_t *path, int32_t *out_tok, int32_t *new_len,
                         int32_t *dev_status, void *stream);

/*
 * KV compaction (Sec. 4.1: the KV cache is the running context).  For every
 * layer l < L, sequence b and k < n_acc[b]: cache slot len[b] + k (through the
 * block table) receives tree row path[b][k], all KV heads, K and V, byte for
 * byte.  Nothing else in any cache changes.  One launch covers all layers.
 *   layers        : host array [L] of cache descriptors
 *   k_tree_layers,
 *   v_tree_layers : host arrays [L] of dev pointers, bf16 [B][T_max][Hkv][D]
 *   n_acc, path   : dev, as produced by sd_accept_tree
 * The tree buffers must not alias the caches.  A destination block outside
 * [0, num_blocks) or a path entry outside [0, T_max) stores SD_ERR_BOUNDS and
 * skips that row.
 */
sd_status sd_compact_kv(const sd_batch *batch, const sd_kv_layer *layers, int32_t L,
                        const void *const *k_tree_layers, const void *const *v_tree_layers,
                        const int32_t *n_acc, const int32_t *path,
                        int32_t *dev_status, void *stream);

/*
 * LM head, acceptance and compaction in one call (Sec. 1: validation ends with the
 * target's tokens deciding which drafts survive; Sec. 4.1: the survivors' KV joins
 * the context).  Equivalent, output for output and byte for byte, to
 *     sd_lmhead_argmax(hidden, W, M = B * T_max, ...)      row b * T_max + i = node i of sequence b
 *     sd_accept_tree(batch, draft_tok, argmax, ...)
 *     sd_compact_kv(batch, layers, L, ..., n_acc, path)
 * but after the LM-head tiles a single kernel (one CTA per sequence and layer;
 * every CTA repeats the merge and the acceptance of its sequence, the CTAs of
 * layer 0 write the outputs) merges the arg-max candidates, picks the accepted path and copies the accepted K/V rows,
 * instead of three launches of a few microseconds each.  Arguments as in the three
 * calls; argmax [B * T_max] and maxlogit (nullable) are outputs as well.
 * B * T_max > 512 or L > 64 falls back to the three separate steps internally.
 */
sd_status sd_lmhead_accept_compact(const sd_batch *batch, const void *hidden, const void *W,
                                   int32_t Hd, int32_t V, const int32_t *draft_tok,
                                   const sd_kv_layer *layers, int32_t L,
                                   const void *const *k_tree_layers, const void *const *v_tree_layers,
                                   int32_t *argmax, float *maxlogit,
                                   int32_t *n_acc, int32_t *path, int32_t *out_tok, int32_t *new_len,
                                   void *workspace, size_t workspace_bytes,
                                   int32_t *dev_status, void *stream);

/*
 * LM head with soft-max statistics, for verification at a sampling temperature
 * (Sec. 1: the drafts are validated by the target model without changing its
 * output distribution; the speculative-sampling rule the paper builds on
 * compares a draft's probability under the target with a uniform number).
 * As sd_lmhead_argmax, plus
 *   lse[r] = log sum_v exp(logits[r][v] * inv_temp)        (natural log, fp32)
 * accumulated in the same epilogue (running reference and sum per row; logits
 * still never reach memory).  argmax and maxlogit may be NULL.
 *   inv_temp    : 1 / temperature, > 0
 *   group_stats : NULL, or dev f32 [ceil(V / 32)][M][2], 8-byte aligned: for every 32
 *                 consecutive vocabulary rows g and hidden row r the pair (largest
 *                 logit of the group, sum over the group of exp((logit - largest) *
 *                 inv_temp)).  sd_accept_tree_sampled uses it to draw its last token
 *                 without reading W a second time.
 *   workspace   : at least sd_workspace_bytes(NULL, M, V)
 */
sd_status sd_lmhead_stats(const void *hidden, const void *W, int32_t M, int32_t Hd, int32_t V,
                          float inv_temp, int32_t *argmax, float *maxlogit, float *lse,
                          float *group_stats, void *workspace, size_t workspace_bytes,
                          int32_t *dev_status, void *stream);

/*
 * sd_lmhead_stats that also keeps the raw logits (Sec. 1 / Sec. 4.2: chain decoding,
 * where a step verifies few rows).  For M rows the logits are M x V floats - 53 MB for
 * root + 10 drafts of 8 sequences at V = 152064, a twentieth of W - and keeping them
 * lets sd_accept_chain_sampled draw its last token without streaming W again.
 *   logits : dev f32 [M][V], logits[r][v] = sum_k hidden[r][k] * W[v][k] (fp32 accumulation)
 * Everything else as sd_lmhead_stats (no group table).
 */
sd_status sd_lmhead_stats_logits(const void *hidden, const void *W, int32_t M, int32_t Hd, int32_t V,
                                 float inv_temp, int32_t *argmax, float *maxlogit, float *lse,
                                 float *logits, void *workspace, size_t workspace_bytes,
                                 int32_t *dev_status, void *stream);

/*
 * Acceptance at a sampling temperature for a deterministically drafted tree
 * (Sec. 1, lossless validation; rule of the cited speculative-sampling work with
 * a point-mass draft distribution).  With p_i = softmax(logits_i * inv_temp) the
 * target distribution at node i:
 *   at node i, residual mass R = 1; for every child c of i in node order:
 *       accept c  iff  u[b][c] * R < p_i(draft_tok[c]);  continue at c with R = 1
 *       otherwise R -= p_i(draft_tok[c])
 *   where no child is accepted the walk stops and one more token is drawn from
 *   p_i restricted to the tokens that are not drafted children of i: the first
 *   token, in vocabulary order, at which the cumulative remaining mass reaches
 *   w[b] times the total remaining mass.
 * Outputs as sd_accept_tree (out_tok = accepted drafts, then the drawn token).
 * All random numbers are inputs: u dev f32 [B][T_max] in [0,1), w dev f32 [B].
 *   hidden, W, Hd, V : the LM head's operands (row b * T_max + i = node i of sequence b)
 *   lse              : dev f32 [B * T_max] from sd_lmhead_stats with the same inv_temp
 *   group_stats      : the table sd_lmhead_stats filled in the same call as lse, or NULL.
 *                      With it the last token is found from the per-group masses and
 *                      32 recomputed logits; without it the stop nodes' rows go
 *                      through the LM head once more and their probabilities over
 *                      the vocabulary (B x V floats, in the workspace) are the only
 *                      logits-sized data that reach memory
 *   workspace        : at least sd_workspace_bytes(batch, B * T_max, V)
 * Siblings must carry distinct tokens (a repeated token among the children the
 * walk looks at stores SD_ERR_INVALID_ARG).  Arithmetic: fp32; a comparison whose
 * two sides differ by less than rounding may fall either way.  A draft token
 * outside [0, V) stores SD_ERR_BOUNDS, a bad tree SD_ERR_INVALID_TREE.
 */
sd_status sd_accept_tree_sampled(const sd_batch *batch, const void *hidden, const void *W,
                                 int32_t Hd, int32_t V, float inv_temp, const float *lse,
                                 const float *group_stats,
                                 const int32_t *draft_tok, const float *u, const float *w,
                                 int32_t *n_acc, int32_t *path, int32_t *out_tok, int32_t *new_len,
                                 void *workspace, size_t workspace_bytes,
                                 int32_t *dev_status, void *stream);

/*
 * Acceptance at a sampling temperature for CHAINS whose tokens were drawn from the
 * draft model's own distributions (Sec. 1, lossless validation; the cited
 * speculative-sampling rule in its general form).  Every tree must be a chain
 * (parents[b][j] == j - 1).  With p_i = softmax(logits_i * inv_temp) the target's and
 * q_i the draft's distribution behind node i (node i + 1's token was drawn from q_i):
 *   walking down from the root, node j is accepted iff
 *       u[b][j] * q_{j-1}(draft_tok[j]) < p_{j-1}(draft_tok[j])          (probability min(1, p/q))
 *   at the first rejection, behind node i = j - 1, one token is drawn from the
 *   normalised positive part of p_i - q_i; if every draft is accepted, from p_leaf:
 *   the first token, in vocabulary order, at which the cumulative mass reaches
 *   w[b] times the total mass.
 * Outputs as sd_accept_tree (path[b][k] = k; out_tok = accepted drafts, then the drawn token).
 *   lse    : dev f32 [B * T_max] from sd_lmhead_stats with the same inv_temp
 *   logits : NULL, or dev f32 [B * T_max][V] as sd_lmhead_stats_logits left them in the same
 *            pass as lse: the stop rows' probabilities are then formed from them and W is
 *            not read a second time
 *   q_tok  : dev f32 [B][T_max], q_tok[b][j] = q_{j-1}(draft_tok[b][j]) for j >= 1
 *   q_rows : dev f32 [B][T_max][V], row [b][i] = q_i; only the row of the node where a
 *            sequence's walk stops is read, and only if a draft was rejected there
 *   u, w   : dev f32 [B][T_max] and [B], uniform numbers in [0, 1)
 *   workspace : at least sd_workspace_bytes(batch, B * T_max, V)
 * Without `logits` the stop nodes' rows go through the LM head once more (their
 * probabilities over the vocabulary, B x V floats in the workspace, are then the only
 * logits-sized data that reach memory).  A tree that branches stores SD_ERR_UNSUPPORTED, a bad tree
 * SD_ERR_INVALID_TREE, a draft token outside [0, V) SD_ERR_BOUNDS (through
 * *dev_status; n_acc[b] = 0 for the first two).  V > 1048576 returns SD_ERR_UNSUPPORTED
 * before anything is launched.  Trees that branch and were sampled from a
 * distribution go through sd_accept_tree_sampled_q, deterministic (top-k) trees
 * through sd_accept_tree_sampled.
 */
sd_status sd_accept_chain_sampled(const sd_batch *batch, const void *hidden, const void *W,
                                  int32_t Hd, int32_t V, float inv_temp, const float *lse,
                                  const float *logits,
                                  const int32_t *draft_tok, const float *q_tok, const float *q_rows,
                                  const float *u, const float *w,
                                  int32_t *n_acc, int32_t *path, int32_t *out_tok, int32_t *new_len,
                                  void *workspace, size_t workspace_bytes,
                                  int32_t *dev_status, void *stream);

/*
 * Acceptance at a sampling temperature for TREES whose children were sampled: every
 * child of node i drawn independently from the draft's distribution q_i (Sec. 1,
 * lossless validation; the cited rule applied child after child).  At node i, with
 * r = p_i = softmax(logits_i * inv_temp):
 *   for every child c of i in node order, x = draft_tok[c]:
 *       accept c  iff  u[b][c] * q_i(x) < r(x);  continue at c with r = p_c
 *       otherwise r <- normalised positive part of r - q_i
 *   where no child is accepted one token is drawn from r: the first token, in
 *   vocabulary order, at which the cumulative mass reaches w[b] times the total.
 * Sibling tokens may repeat.  A chain is the special case of one child per node.
 *   lse, logits : dev f32 [B * T_max] and [B * T_max][V] from sd_lmhead_stats_logits
 *                 with the same inv_temp (row b * T_max + i = node i of sequence b)
 *   q_rows      : dev f32 [B][T_max][V], row [b][i] = q_i (rows of nodes the walk visits are read)
 *   u, w        : dev f32 [B][T_max] and [B], uniform numbers in [0, 1)
 * Outputs as sd_accept_tree.  One cluster of eight CTAs per sequence keeps p_i and q_i
 * of the current node in shared memory (V <= 163840, else SD_ERR_UNSUPPORTED before
 * anything is launched); every rejection costs one reduction over the vocabulary.
 * A bad tree stores SD_ERR_INVALID_TREE, a draft token outside [0, V) SD_ERR_BOUNDS
 * (n_acc[b] = 0 in both cases).  Arithmetic: fp32, sums in a fixed order.
 */
sd_status sd_accept_tree_sampled_q(const sd_batch *batch, int32_t V, float inv_temp,
                                   const float *lse, const float *logits,
                                   const int32_t *draft_tok, const float *q_rows,
                                   const float *u, const float *w,
                                   int32_t *n_acc, int32_t *path, int32_t *out_tok, int32_t *new_len,
                                   int32_t *dev_status, void *stream);

/*
 * LM head, acceptance at a sampling temperature and compaction in one call (Sec. 1:
 * lossless validation; Sec. 4.1: the survivors' KV joins the context).  Equivalent,
 * output for output and byte for byte, to
 *     sd_lmhead_stats(hidden, W, M = B * T_max, ..., argmax = NULL, maxlogit = NULL, lse, group_stats)
 *     sd_accept_tree_sampled(batch, hidden, W, ..., lse, group_stats, draft_tok, u, w, ...)
 *     sd_compact_kv(batch, layers, L, ..., n_acc, path)
 * but behind the LM-head tiles a single kernel does the rest: one cluster of eight
 * CTAs per sequence merges the rows' soft-max statistics, computes the drafted
 * tokens' probabilities, walks the tree, draws the last token from the group table
 * and copies the accepted K/V rows (each CTA a share of the layers) - two launches
 * instead of six.  Arguments as in the three calls:
 *   lse         : dev f32 [B * T_max], output
 *   group_stats : dev f32 [ceil(V / 32)][B * T_max][2], 8-byte aligned, scratch that the
 *                 call fills and reads (required here)
 *   workspace   : at least sd_workspace_bytes(batch, B * T_max, V)
 * V > 262144 returns SD_ERR_UNSUPPORTED before anything is launched; B * T_max > 512
 * or L > 64 falls back to the separate steps internally.
 */
sd_status sd_lmhead_accept_sampled_compact(const sd_batch *batch, const void *hidden, const void *W,
                                           int32_t Hd, int32_t V, float inv_temp,
                                           const int32_t *draft_tok, const float *u, const float *w,
                                           const sd_kv_layer *layers, int32_t L,
                                           const void *const *k_tree_layers, const void *const *v_tree_layers,
                                           float *lse, float *group_stats,
                                           int32_t *n_acc, int32_t *path, int32_t *out_tok, int32_t *new_len,
                                           void *workspace, size_t workspace_bytes,
                                           int32_t *dev_status, void *stream);

/*
 * Draft-side feature aggregation (Sec. 3.1.1, f_c^i = Flatten(CrossAttention(f_q, f_i, f_i))):
 * Q meta queries, shared by all tokens, attend over the L target-layer features
 * of every token.  This is the attention core for H heads of size 128
 * (D = H * 128); the module's projections are ordinary GEMMs outside it:
 *   for token i, head h:  p = softmax_l(scale * <qp[q, h], k[i, l, h]>),
 *                         out[i, q, h] = sum_l p[q, l] * v[i, l, h]
 *   qp  : dev bf16 [Q][D]      projected meta queries (the same for every token)
 *   k,v : dev bf16 [S][L][D]   the tokens' (projected) layer features; may be the same buffer
 *   out : dev bf16 [S][Q][D]   = [S][Q * D] flattened, as the paper uses it
 * L <= 32, Q <= 8.  fp32 accumulation, bf16 output (round to nearest even).
 * Every K and V row is read once; the call is bound by HBM bandwidth.
 */
sd_status sd_draft_feature_attention(const void *qp, const void *k, const void *v,
                                     int32_t S, int32_t L, int32_t Q, int32_t H, int32_t D,
                                     float scale, void *out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SDVERIFY_H */
