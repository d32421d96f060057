// Tree bookkeeping kernels: ancestor masks and greedy acceptance.
// Integer work only; one warp per sequence.
#include "common.cuh"

namespace sdv {

// anc_mask[b][i] = bit i | anc_mask[b][parent(i)], computed by walking up.
__global__ void tree_prepare_kernel(sd_batch bt, int32_t* status) {
    const int b = blockIdx.x;
    const int lane = threadIdx.x;
    const int T = bt.T_max;
    const int n = bt.n_nodes[b];
    const int32_t* par = bt.parents + (size_t)b * T;
    uint64_t* am = bt.anc_mask + (size_t)b * T;
    if (n < 1 || n > T) {
        if (lane == 0) set_status(status, SD_ERR_INVALID_TREE);
        return;
    }
    // validate first so that the walks below are bounded and in range
    bool bad = false;
    for (int i = lane; i < n; i += 32) {
        int p = par[i];
        if (i == 0 ? (p != -1) : (p < 0 || p >= i)) bad = true;
    }
    if (__any_sync(0xffffffffu, bad)) {
        if (lane == 0) set_status(status, SD_ERR_INVALID_TREE);
        return;
    }
    for (int i = lane; i < T; i += 32) {
        uint64_t m = 0;
        if (i < n) {
            int j = i;
            for (int step = 0; step < kMaxT && j >= 0; ++step) {
                m |= 1ull << j;
                j = par[j];
            }
        }
        am[i] = m;
    }
}

// Greedy acceptance: each lane scores the root paths of up to two nodes,
// the warp picks the deepest valid one (smallest index among equals).
__global__ void accept_kernel(sd_batch bt, const int32_t* __restrict__ draft,
                              const int32_t* __restrict__ target,
                              int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                              int32_t* status) {
    const int b = blockIdx.x;
    const int lane = threadIdx.x;
    const int T = bt.T_max;
    const int n = bt.n_nodes[b];
    const int32_t* par = bt.parents + (size_t)b * T;
    const int32_t* dt = draft + (size_t)b * T;
    const int32_t* tg = target + (size_t)b * T;
    bool bad = (n < 1 || n > T);
    if (!bad)
        for (int i = lane; i < n; i += 32) {
            int p = par[i];
            if (i == 0 ? (p != -1) : (p < 0 || p >= i)) bad = true;
        }
    if (__any_sync(0xffffffffu, bad)) {
        if (lane == 0) set_status(status, SD_ERR_INVALID_TREE);
        return;
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
            if (k >= 1) ot[k - 1] = dt[j];
            j = par[j];
        }
        ot[na - 1] = tg[best];
    }
}

sd_status launch_tree_prepare(const sd_batch& bt, int32_t* dev_status, cudaStream_t st) {
    tree_prepare_kernel<<<bt.B, 32, 0, st>>>(bt, dev_status);
    return cuda_ok(cudaGetLastError());
}

sd_status launch_accept(const sd_batch& bt, const int32_t* draft, const int32_t* target,
                        int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                        int32_t* dev_status, cudaStream_t st) {
    accept_kernel<<<bt.B, 32, 0, st>>>(bt, draft, target, n_acc, path, out_tok, new_len, dev_status);
    return cuda_ok(cudaGetLastError());
}

}  // namespace sdv
