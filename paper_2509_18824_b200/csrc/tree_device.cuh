// Device-side pieces shared by the stand-alone kernels (acceptance, compaction, LM-head merge) and
// the fused tail kernel that runs the three back to back for one sequence per CTA.
#pragma once
#include "common.cuh"

namespace sdv {

constexpr int kLayersPerLaunch = 64;     // layer descriptors travel as kernel parameters
constexpr int kLmMaxCols = 512;          // hidden rows per LM-head pass = row stride of the candidate tables

struct CompactLayers {
    uint4* kc[kLayersPerLaunch];
    uint4* vc[kLayersPerLaunch];
    const uint4* kt[kLayersPerLaunch];
    const uint4* vt[kLayersPerLaunch];
    int32_t num_blocks[kLayersPerLaunch];
};

// descriptors of layers [l0, l0 + nl) (implemented beside the compaction kernel)
void fill_compact_layers(CompactLayers* ly, const sd_kv_layer* layers, const void* const* kt, const void* const* vt,
                         int l0, int nl);

__device__ __forceinline__ float key_to_float(int32_t k) {
    return __int_as_float(k < 0 ? (k ^ 0x7fffffff) : k);
}

// (key, index) candidates: larger key wins, lower index among equal keys
__device__ __forceinline__ void take_better(int32_t& k, int32_t& i, int32_t k2, int32_t i2) {
    if (k2 > k || (k2 == k && i2 < i)) { k = k2; i = i2; }
}

__device__ __forceinline__ float ex2_lm(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// running (reference, sum) of a row's soft-max statistics takes in a new partial (ref2, sum2):
// sum counts 2^((logit - ref) * c2)
__device__ __forceinline__ void merge_sumexp(float& ref, float& sum, float ref2, float sum2, float c2) {
    if (!(sum2 > 0.f)) return;
    if (ref2 > ref) { sum = sum * ex2_lm((ref - ref2) * c2) + sum2; ref = ref2; }
    else            { sum += sum2 * ex2_lm((ref2 - ref) * c2); }
}

// Candidates and soft-max partials of one hidden row (column `col` of the per-CTA tables), merged by the
// eight consecutive lanes that share the row: lane `sub` takes the CTAs sub, sub + 8, ..., then three
// exchange steps combine the eight (always lower lane first, so all eight end with the same bits).
// Every lane of the warp must call this; rows beyond the problem pass active = false.  Returns the
// row's log sum exp(logit / temperature) (natural log); k, i: the arg-max candidate (key, index).
__device__ __forceinline__ float merge_row_stats(const int32_t* __restrict__ part_key, const int32_t* __restrict__ part_idx,
                                                 const float* __restrict__ part_ref, const float* __restrict__ part_sum,
                                                 int n_ctas, int row_stride, int col, bool active, int sub, float c2,
                                                 int32_t& k, int32_t& i) {
    k = INT32_MIN; i = 0x7fffffff;
    float rf = -INFINITY, sm = 0.f;
    if (active) {
        // (the loads of a batch are issued together, then merged in CTA order: latency-bound)
        constexpr int kAhead = 20;                  // 148 CTAs: 19 per lane
        for (int c0 = sub; c0 < n_ctas; c0 += 8 * kAhead) {
            int32_t pk[kAhead], pi[kAhead];
            float pr[kAhead], ps[kAhead];
#pragma unroll
            for (int a = 0; a < kAhead; ++a) {
                const int c = c0 + 8 * a;
                if (c < n_ctas) {
                    pk[a] = __ldg(part_key + (size_t)c * row_stride + col);
                    pi[a] = __ldg(part_idx + (size_t)c * row_stride + col);
                    pr[a] = __ldg(part_ref + (size_t)c * row_stride + col);
                    ps[a] = __ldg(part_sum + (size_t)c * row_stride + col);
                }
            }
#pragma unroll
            for (int a = 0; a < kAhead; ++a)
                if (c0 + 8 * a < n_ctas) {
                    take_better(k, i, pk[a], pi[a]);
                    merge_sumexp(rf, sm, pr[a], ps[a], c2);
                }
        }
    }
#pragma unroll
    for (int d = 1; d <= 4; d <<= 1) {
        const int32_t k2 = __shfl_xor_sync(0xffffffffu, k, d), i2 = __shfl_xor_sync(0xffffffffu, i, d);
        const float rf2 = __shfl_xor_sync(0xffffffffu, rf, d), sm2 = __shfl_xor_sync(0xffffffffu, sm, d);
        take_better(k, i, k2, i2);
        float ra = (sub & d) ? rf2 : rf, sa = (sub & d) ? sm2 : sm;
        const float rb = (sub & d) ? rf : rf2, sb = (sub & d) ? sm : sm2;
        merge_sumexp(ra, sa, rb, sb, c2);
        rf = ra; sm = sa;
    }
    return (rf * c2 + log2f(sm)) * 0.6931471805599453f;
}

// Greedy acceptance for one sequence, executed by one warp.  par/dt/tg point at the sequence's
// parents, draft tokens and target arg-max (tg may be shared memory).  Returns the number of
// accepted nodes (0 for a bad tree, which is reported through *status) and, in lane 0, has written
// n_acc, new_len, path and out_tok; `path_out` (nullable, e.g. shared memory) receives the path too.
__device__ __forceinline__ int accept_sequence(const sd_batch& bt, int b, int lane, const int32_t* par,
                                               const int32_t* dt, const int32_t* tg,
                                               int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                                               int32_t* path_out, int32_t* status) {
    const int T = bt.T_max;
    const int n = bt.n_nodes[b];
    bool bad = (n < 1 || n > T);
    if (!bad)
        for (int i = lane; i < n; i += 32) {
            int p = par[i];
            if (i == 0 ? (p != -1) : (p < 0 || p >= i)) bad = true;
        }
    if (__any_sync(0xffffffffu, bad)) {
        if (lane == 0) set_status(status, SD_ERR_INVALID_TREE);
        return 0;
    }
    // key = depth * 64 + (63 - index) for valid nodes: max key = deepest, lowest index
    int best_key = -1;
    for (int i = lane; i < n; i += 32) {
        bool ok = true;
        int depth = 0;
        int j = i;
        for (int step = 0; step < kMaxT && j > 0; ++step) {
            int p = par[j];
            ok = ok && (dt[j] == tg[p]);
            ++depth;
            j = p;
        }
        if (ok) best_key = max(best_key, depth * 64 + (63 - i));
    }
    best_key = __reduce_max_sync(0xffffffffu, best_key);   // node 0 is always valid
    const int best = 63 - (best_key & 63);
    const int na = (best_key >> 6) + 1;
    int32_t* pa = path + (size_t)b * T;
    int32_t* ot = out_tok + (size_t)b * T;
    for (int k = na + lane; k < T; k += 32) { pa[k] = -1; ot[k] = -1; }
    if (lane == 0) {
        n_acc[b] = na;
        new_len[b] = bt.len[b] + na;
        int j = best;
        for (int k = na - 1; k >= 0; --k) {
            pa[k] = j;
            if (path_out) path_out[k] = j;
            if (k >= 1) ot[k - 1] = dt[j];
            j = par[j];
        }
        ot[na - 1] = tg[best];
    }
    return na;
}

// Copies the accepted rows of sequence b in layers [l0, l0 + n_layers): work items idx = tid, tid + stride, ...
// One item = one 16-byte vector of one (layer, accepted node, K or V, KV head).  `path` holds the
// sequence's accepted nodes (global or shared memory).
__device__ __forceinline__ void compact_sequence(const sd_batch& bt, const CompactLayers& ly, int l0, int n_layers, int b,
                                                 int na, const int32_t* path, int tid, int stride,
                                                 int32_t* status) {
    const int T = bt.T_max;
    const int len = bt.len[b];
    const int vec_per_head = bt.D * 2 / 16;               // 16 for D = 128
    const int vec_per_node = bt.Hkv * vec_per_head;       // per K or V
    const int per_layer = na * 2 * vec_per_node;
    const int total = per_layer * n_layers;
    const int per_node = 2 * vec_per_node;                 // K and V vectors of one node
    if (stride % per_node == 0) {
        // Every thread keeps its place inside a node (K or V, head, 16-byte piece) and only walks over
        // the accepted nodes and the layers: no index arithmetic beyond the two table look-ups per vector.
        const int sub = tid % per_node;
        const int is_v = sub / vec_per_node;
        const int kvh = (sub - is_v * vec_per_node) / vec_per_head;
        const int c = sub - is_v * vec_per_node - kvh * vec_per_head;
        const int k_step = stride / per_node;
        constexpr int kUnroll = 4;                         // nodes in flight per thread: loads before stores
        for (int k0 = tid / per_node; k0 < na; k0 += k_step * kUnroll) {
            size_t src[kUnroll], dst[kUnroll];
            int blk[kUnroll];
            bool has[kUnroll];                             // this slot holds an accepted node
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int k = k0 + u * k_step;
                blk[u] = -1;
                has[u] = false;
                if (k >= na) continue;
                const int node = path[k];
                const int t = len + k;
                if (node < 0 || node >= T || t < 0 || t / kBlock >= bt.max_blocks_per_seq) {
                    set_status(status, SD_ERR_BOUNDS);
                    continue;
                }
                has[u] = true;
                blk[u] = bt.block_table[(size_t)b * bt.max_blocks_per_seq + t / kBlock];
                src[u] = (((size_t)b * T + node) * bt.Hkv + kvh) * vec_per_head + c;
                dst[u] = (((size_t)(blk[u] < 0 ? 0 : blk[u]) * bt.Hkv + kvh) * kBlock + (t % kBlock)) * vec_per_head + c;
            }
            for (int l = l0; l < l0 + n_layers; ++l) {
                const uint4* from = is_v ? ly.vt[l] : ly.kt[l];
                uint4* to = is_v ? ly.vc[l] : ly.kc[l];
                const int nb = ly.num_blocks[l];
                uint4 val[kUnroll];
                bool live[kUnroll];
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    live[u] = has[u] && blk[u] >= 0 && blk[u] < nb;
                    if (has[u] && !live[u]) set_status(status, SD_ERR_BOUNDS);
                    if (live[u]) val[u] = from[src[u]];
                }
#pragma unroll
                for (int u = 0; u < kUnroll; ++u)
                    if (live[u]) to[dst[u]] = val[u];
            }
        }
        return;
    }
    for (int idx = tid; idx < total; idx += stride) {
        const int li = idx / per_layer;
        const int l = l0 + li;
        int rem = idx - li * per_layer;
        const int k = rem / (2 * vec_per_node);
        rem -= k * 2 * vec_per_node;
        const int is_v = rem / vec_per_node;
        rem -= is_v * vec_per_node;
        const int kvh = rem / vec_per_head;
        const int c = rem - kvh * vec_per_head;
        const int node = path[k];
        const int t = len + k;
        if (node < 0 || node >= T || t < 0 || t / kBlock >= bt.max_blocks_per_seq) {
            set_status(status, SD_ERR_BOUNDS);
            continue;
        }
        const int blk = bt.block_table[(size_t)b * bt.max_blocks_per_seq + t / kBlock];
        if (blk < 0 || blk >= ly.num_blocks[l]) {
            set_status(status, SD_ERR_BOUNDS);
            continue;
        }
        const size_t src = (((size_t)b * T + node) * bt.Hkv + kvh) * vec_per_head + c;
        const size_t dst = (((size_t)blk * bt.Hkv + kvh) * kBlock + (t % kBlock)) * vec_per_head + c;
        if (is_v) ly.vc[l][dst] = ly.vt[l][src];
        else      ly.kc[l][dst] = ly.kt[l][src];
    }
}

}  // namespace sdv
