// C-ABI entry points: argument validation, then the kernel launchers.
#include "common.cuh"

#include <stdlib.h>

using namespace sdv;

namespace sdv {
TestKnobs test_knobs() {
    TestKnobs k{1ll << 31, 0, 0};
    if (const char* e = getenv("SDV_TEST_WAIT_CYCLES")) { const long long v = atoll(e); if (v >= 1000) k.wait_cycles = v; }
    if (const char* e = getenv("SDV_TEST_WITHHOLD")) k.withhold = atoi(e) == 1 ? 1 : 0;
    if (const char* e = getenv("SDV_TEST_CHUNKS")) { const int v = atoi(e); if (v == 1 || v == 2 || v == 4 || v == 8) k.chunks = v; }
    return k;
}
}  // namespace sdv

namespace {

sd_status check_geometry(const sd_batch* bt, bool need_pointers) {
    if (!bt) return SD_ERR_INVALID_ARG;
    if (bt->B < 1 || bt->T_max < 1 || bt->Hq < 1 || bt->Hkv < 1 || bt->max_blocks_per_seq < 1)
        return SD_ERR_INVALID_ARG;
    if (bt->D != kD || bt->block_size != kBlock || bt->T_max > kMaxT) return SD_ERR_UNSUPPORTED;
    if (bt->Hq % bt->Hkv != 0 || bt->Hq / bt->Hkv > 8) return SD_ERR_UNSUPPORTED;
    if (need_pointers) {
        if (!bt->block_table || !bt->len || !bt->n_nodes || !bt->parents) return SD_ERR_INVALID_ARG;
        if (!aligned16(bt->block_table) || !aligned16(bt->len) || !aligned16(bt->n_nodes) ||
            !aligned16(bt->parents))
            return SD_ERR_INVALID_ARG;
    }
    return SD_OK;
}

bool ok_ptr(const void* p) { return p && aligned16(p); }

}  // namespace

extern "C" {

int sd_version(void) { return 100; }

const char* sd_status_string(sd_status s) {
    switch (s) {
        case SD_OK: return "SD_OK";
        case SD_ERR_INVALID_ARG: return "SD_ERR_INVALID_ARG";
        case SD_ERR_INVALID_TREE: return "SD_ERR_INVALID_TREE";
        case SD_ERR_UNSUPPORTED: return "SD_ERR_UNSUPPORTED";
        case SD_ERR_WORKSPACE: return "SD_ERR_WORKSPACE";
        case SD_ERR_CUDA: return "SD_ERR_CUDA";
        case SD_ERR_TIMEOUT: return "SD_ERR_TIMEOUT";
        case SD_ERR_BOUNDS: return "SD_ERR_BOUNDS";
    }
    return "SD_ERR_UNKNOWN";
}

size_t sd_workspace_bytes(const sd_batch* geom, int32_t M, int32_t V) {
    size_t a = 0, l = 0;
    if (geom && check_geometry(geom, false) == SD_OK) a = attention_workspace_bytes(*geom);
    if (M > 0 && V > 0) l = stats_workspace_bytes(M, V);    // covers sd_lmhead_argmax, the fused tail and sd_lmhead_stats
    if (geom && V > 0 && check_geometry(geom, false) == SD_OK) {
        const size_t sw = sampled_workspace_bytes(geom->B, geom->T_max, V, 16384);   // sd_accept_tree_sampled (Hd <= 16384)
        if (sw > l) l = sw;
    }
    size_t n = a > l ? a : l;
    return (n + 255) & ~(size_t)255;
}

sd_status sd_tree_prepare(const sd_batch* batch, int32_t* dev_status, void* stream) {
    sd_status s = check_geometry(batch, true);
    if (s != SD_OK) return s;
    if (!ok_ptr(batch->anc_mask) || !dev_status) return SD_ERR_INVALID_ARG;
    return launch_tree_prepare(*batch, dev_status, static_cast<cudaStream_t>(stream));
}

sd_status sd_verify_attention(const sd_batch* batch, const sd_kv_layer* cache,
                              const void* q, const void* k_tree, const void* v_tree,
                              float scale, void* out, float* lse,
                              void* workspace, size_t workspace_bytes,
                              int32_t* dev_status, void* stream) {
    sd_status s = check_geometry(batch, true);
    if (s != SD_OK) return s;
    if (!cache || !ok_ptr(cache->k) || !ok_ptr(cache->v) || cache->num_blocks < 1) return SD_ERR_INVALID_ARG;
    if (!ok_ptr(q) || !ok_ptr(k_tree) || !ok_ptr(v_tree) || !ok_ptr(out) || !ok_ptr(batch->anc_mask))
        return SD_ERR_INVALID_ARG;
    if (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)) return SD_ERR_INVALID_ARG;
    if (!ok_ptr(workspace) || !dev_status) return SD_ERR_INVALID_ARG;
    if (!(scale > 0.f)) return SD_ERR_INVALID_ARG;
    return launch_attention(*batch, *cache, q, k_tree, v_tree, scale, out, lse, workspace,
                            workspace_bytes, dev_status, static_cast<cudaStream_t>(stream));
}

sd_status sd_verify_attention_layers(const sd_batch* batch, const sd_kv_layer* caches, int32_t L,
                                     const void* const* q_layers, const void* const* k_tree_layers,
                                     const void* const* v_tree_layers, float scale,
                                     void* const* out_layers, float* const* lse_layers,
                                     void* workspace, size_t workspace_bytes,
                                     int32_t* dev_status, void* stream) {
    sd_status s = check_geometry(batch, true);
    if (s != SD_OK) return s;
    if (!caches || L < 1 || !q_layers || !k_tree_layers || !v_tree_layers || !out_layers) return SD_ERR_INVALID_ARG;
    if (!ok_ptr(batch->anc_mask) || !ok_ptr(workspace) || !dev_status) return SD_ERR_INVALID_ARG;
    if (!(scale > 0.f)) return SD_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l) {
        if (!ok_ptr(caches[l].k) || !ok_ptr(caches[l].v) || caches[l].num_blocks < 1) return SD_ERR_INVALID_ARG;
        if (!ok_ptr(q_layers[l]) || !ok_ptr(k_tree_layers[l]) || !ok_ptr(v_tree_layers[l]) || !ok_ptr(out_layers[l]))
            return SD_ERR_INVALID_ARG;
        if (lse_layers && lse_layers[l] && (reinterpret_cast<uintptr_t>(lse_layers[l]) & 3u)) return SD_ERR_INVALID_ARG;
    }
    if (workspace_bytes < attention_workspace_bytes(*batch)) return SD_ERR_WORKSPACE;
    return launch_attention_layers(*batch, caches, L, q_layers, k_tree_layers, v_tree_layers, scale, out_layers,
                                   lse_layers, dev_status, static_cast<cudaStream_t>(stream));
}

sd_status sd_lmhead_argmax(const void* hidden, const void* W, int32_t M, int32_t Hd, int32_t V,
                           int32_t* argmax, float* maxlogit, void* workspace, size_t workspace_bytes,
                           int32_t* dev_status, void* stream) {
    if (!ok_ptr(hidden) || !ok_ptr(W) || !argmax || !ok_ptr(workspace) || !dev_status) return SD_ERR_INVALID_ARG;
    if (M < 1 || V < 1 || Hd < 1) return SD_ERR_INVALID_ARG;
    if (Hd % 64 != 0) return SD_ERR_UNSUPPORTED;
    return launch_lmhead(hidden, W, M, Hd, V, argmax, maxlogit, workspace, workspace_bytes, dev_status,
                         static_cast<cudaStream_t>(stream));
}

sd_status sd_accept_tree(const sd_batch* batch, const int32_t* draft_tok, const int32_t* target_argmax,
                         int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                         int32_t* dev_status, void* stream) {
    sd_status s = check_geometry(batch, true);
    if (s != SD_OK) return s;
    if (!draft_tok || !target_argmax || !n_acc || !path || !out_tok || !new_len || !dev_status)
        return SD_ERR_INVALID_ARG;
    return launch_accept(*batch, draft_tok, target_argmax, n_acc, path, out_tok, new_len, dev_status,
                         static_cast<cudaStream_t>(stream));
}

sd_status sd_compact_kv(const sd_batch* batch, const sd_kv_layer* layers, int32_t L,
                        const void* const* k_tree_layers, const void* const* v_tree_layers,
                        const int32_t* n_acc, const int32_t* path, int32_t* dev_status, void* stream) {
    sd_status s = check_geometry(batch, true);
    if (s != SD_OK) return s;
    if (!layers || L < 1 || !k_tree_layers || !v_tree_layers || !n_acc || !path || !dev_status)
        return SD_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l) {
        if (!ok_ptr(layers[l].k) || !ok_ptr(layers[l].v) || layers[l].num_blocks < 1) return SD_ERR_INVALID_ARG;
        if (!ok_ptr(k_tree_layers[l]) || !ok_ptr(v_tree_layers[l])) return SD_ERR_INVALID_ARG;
    }
    return launch_compact(*batch, layers, L, k_tree_layers, v_tree_layers, n_acc, path, dev_status,
                          static_cast<cudaStream_t>(stream));
}

sd_status sd_lmhead_accept_compact(const sd_batch* batch, const void* hidden, const void* W, int32_t Hd, int32_t V,
                                   const int32_t* draft_tok, const sd_kv_layer* layers, int32_t L,
                                   const void* const* k_tree_layers, const void* const* v_tree_layers,
                                   int32_t* argmax, float* maxlogit,
                                   int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                                   void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream) {
    sd_status s = check_geometry(batch, true);
    if (s != SD_OK) return s;
    if (!ok_ptr(hidden) || !ok_ptr(W) || !argmax || !ok_ptr(workspace) || !dev_status) return SD_ERR_INVALID_ARG;
    if (V < 1 || Hd < 1) return SD_ERR_INVALID_ARG;
    if (Hd % 64 != 0) return SD_ERR_UNSUPPORTED;
    if (!draft_tok || !n_acc || !path || !out_tok || !new_len) return SD_ERR_INVALID_ARG;
    if (!layers || L < 1 || !k_tree_layers || !v_tree_layers) return SD_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l) {
        if (!ok_ptr(layers[l].k) || !ok_ptr(layers[l].v) || layers[l].num_blocks < 1) return SD_ERR_INVALID_ARG;
        if (!ok_ptr(k_tree_layers[l]) || !ok_ptr(v_tree_layers[l])) return SD_ERR_INVALID_ARG;
    }
    return launch_lmhead_accept_compact(*batch, hidden, W, Hd, V, draft_tok, layers, L, k_tree_layers, v_tree_layers,
                                        argmax, maxlogit, n_acc, path, out_tok, new_len, workspace, workspace_bytes,
                                        dev_status, static_cast<cudaStream_t>(stream));
}

sd_status sd_lmhead_stats(const void* hidden, const void* W, int32_t M, int32_t Hd, int32_t V, float inv_temp,
                          int32_t* argmax, float* maxlogit, float* lse, float* group_stats,
                          void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream) {
    if (group_stats && (reinterpret_cast<uintptr_t>(group_stats) & 7u)) return SD_ERR_INVALID_ARG;
    if (!ok_ptr(hidden) || !ok_ptr(W) || !lse || !ok_ptr(workspace) || !dev_status) return SD_ERR_INVALID_ARG;
    if (M < 1 || V < 1 || Hd < 1 || !(inv_temp > 0.f)) return SD_ERR_INVALID_ARG;
    if (Hd % 64 != 0) return SD_ERR_UNSUPPORTED;
    return launch_lmhead_stats(hidden, W, M, Hd, V, inv_temp, argmax, maxlogit, lse, group_stats, workspace,
                               workspace_bytes, dev_status, static_cast<cudaStream_t>(stream));
}

sd_status sd_accept_tree_sampled(const sd_batch* batch, const void* hidden, const void* W, int32_t Hd, int32_t V,
                                 float inv_temp, const float* lse, const float* group_stats, const int32_t* draft_tok,
                                 const float* u, const float* w,
                                 int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                                 void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream) {
    sd_status s = check_geometry(batch, true);
    if (s != SD_OK) return s;
    if (!ok_ptr(hidden) || !ok_ptr(W) || !lse || !draft_tok || !u || !w) return SD_ERR_INVALID_ARG;
    if (!n_acc || !path || !out_tok || !new_len || !ok_ptr(workspace) || !dev_status) return SD_ERR_INVALID_ARG;
    if (V < 1 || Hd < 1 || !(inv_temp > 0.f)) return SD_ERR_INVALID_ARG;
    if (Hd % 64 != 0) return SD_ERR_UNSUPPORTED;
    return launch_accept_sampled(*batch, hidden, W, Hd, V, inv_temp, lse, group_stats, draft_tok, u, w, n_acc, path, out_tok,
                                 new_len, workspace, workspace_bytes, dev_status, static_cast<cudaStream_t>(stream));
}

sd_status sd_lmhead_stats_logits(const void* hidden, const void* W, int32_t M, int32_t Hd, int32_t V, float inv_temp,
                                 int32_t* argmax, float* maxlogit, float* lse, float* logits,
                                 void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream) {
    if (!ok_ptr(hidden) || !ok_ptr(W) || !lse || !logits || !ok_ptr(workspace) || !dev_status) return SD_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(logits) & 3u) return SD_ERR_INVALID_ARG;
    if (M < 1 || V < 1 || Hd < 1 || !(inv_temp > 0.f)) return SD_ERR_INVALID_ARG;
    if (Hd % 64 != 0) return SD_ERR_UNSUPPORTED;
    return launch_lmhead_stats(hidden, W, M, Hd, V, inv_temp, argmax, maxlogit, lse, nullptr, workspace, workspace_bytes,
                               dev_status, static_cast<cudaStream_t>(stream), logits);
}

sd_status sd_accept_chain_sampled(const sd_batch* batch, const void* hidden, const void* W, int32_t Hd, int32_t V,
                                  float inv_temp, const float* lse, const float* logits,
                                  const int32_t* draft_tok, const float* q_tok,
                                  const float* q_rows, const float* u, const float* w,
                                  int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                                  void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream) {
    sd_status s = check_geometry(batch, true);
    if (s != SD_OK) return s;
    if (!ok_ptr(hidden) || !ok_ptr(W) || !lse || !draft_tok || !q_tok || !q_rows || !u || !w) return SD_ERR_INVALID_ARG;
    if (!n_acc || !path || !out_tok || !new_len || !ok_ptr(workspace) || !dev_status) return SD_ERR_INVALID_ARG;
    if (V < 1 || Hd < 1 || !(inv_temp > 0.f)) return SD_ERR_INVALID_ARG;
    if (Hd % 64 != 0) return SD_ERR_UNSUPPORTED;
    return launch_accept_chain_sampled(*batch, hidden, W, Hd, V, inv_temp, lse, logits, draft_tok, q_tok, q_rows, u, w, n_acc, path,
                                       out_tok, new_len, workspace, workspace_bytes, dev_status,
                                       static_cast<cudaStream_t>(stream));
}

sd_status sd_accept_tree_sampled_q(const sd_batch* batch, int32_t V, float inv_temp, const float* lse, const float* logits,
                                   const int32_t* draft_tok, const float* q_rows, const float* u, const float* w,
                                   int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                                   int32_t* dev_status, void* stream) {
    sd_status s = check_geometry(batch, true);
    if (s != SD_OK) return s;
    if (!lse || !logits || !draft_tok || !q_rows || !u || !w) return SD_ERR_INVALID_ARG;
    if (!n_acc || !path || !out_tok || !new_len || !dev_status) return SD_ERR_INVALID_ARG;
    if (V < 1 || !(inv_temp > 0.f)) return SD_ERR_INVALID_ARG;
    return launch_accept_tree_sampled_q(*batch, V, inv_temp, lse, logits, draft_tok, q_rows, u, w, n_acc, path, out_tok,
                                        new_len, dev_status, static_cast<cudaStream_t>(stream));
}

sd_status sd_lmhead_accept_sampled_compact(const sd_batch* batch, const void* hidden, const void* W, int32_t Hd, int32_t V,
                                           float inv_temp, const int32_t* draft_tok, const float* u, const float* w,
                                           const sd_kv_layer* layers, int32_t L,
                                           const void* const* k_tree_layers, const void* const* v_tree_layers,
                                           float* lse, float* group_stats,
                                           int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                                           void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream) {
    sd_status s = check_geometry(batch, true);
    if (s != SD_OK) return s;
    if (!ok_ptr(hidden) || !ok_ptr(W) || !lse || !group_stats || !draft_tok || !u || !w) return SD_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(group_stats) & 7u) return SD_ERR_INVALID_ARG;
    if (!n_acc || !path || !out_tok || !new_len || !ok_ptr(workspace) || !dev_status) return SD_ERR_INVALID_ARG;
    if (V < 1 || Hd < 1 || !(inv_temp > 0.f)) return SD_ERR_INVALID_ARG;
    if (Hd % 64 != 0) return SD_ERR_UNSUPPORTED;
    if (!layers || L < 1 || !k_tree_layers || !v_tree_layers) return SD_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l) {
        if (!ok_ptr(layers[l].k) || !ok_ptr(layers[l].v) || layers[l].num_blocks < 1) return SD_ERR_INVALID_ARG;
        if (!ok_ptr(k_tree_layers[l]) || !ok_ptr(v_tree_layers[l])) return SD_ERR_INVALID_ARG;
    }
    return launch_lmhead_accept_sampled_compact(*batch, hidden, W, Hd, V, inv_temp, draft_tok, u, w, layers, L, k_tree_layers,
                                                v_tree_layers, lse, group_stats, n_acc, path, out_tok, new_len, workspace,
                                                workspace_bytes, dev_status, static_cast<cudaStream_t>(stream));
}

sd_status sd_draft_feature_attention(const void* qp, const void* k, const void* v, int32_t S, int32_t L, int32_t Q,
                                     int32_t H, int32_t D, float scale, void* out, void* stream) {
    if (!ok_ptr(qp) || !ok_ptr(k) || !ok_ptr(v) || !ok_ptr(out)) return SD_ERR_INVALID_ARG;
    if (S < 1 || L < 1 || Q < 1 || H < 1 || !(scale > 0.f)) return SD_ERR_INVALID_ARG;
    if (D != H * 128 || L > 32 || Q > 8) return SD_ERR_UNSUPPORTED;
    return launch_draft_feature_attention(qp, k, v, S, L, Q, H, scale, out, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
