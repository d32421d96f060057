// Tree bookkeeping kernels: ancestor masks and greedy acceptance.
// Integer work only; one warp per sequence.
#include "tree_device.cuh"

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
    const int T = bt.T_max;
    accept_sequence(bt, b, threadIdx.x, bt.parents + (size_t)b * T, draft + (size_t)b * T, target + (size_t)b * T,
                    n_acc, path, out_tok, new_len, nullptr, status);
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
