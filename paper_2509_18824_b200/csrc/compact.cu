// KV compaction: accepted tree rows gathered into their paged cache slots,
// every layer in one launch, 16-byte vector copies.
#include "common.cuh"

namespace sdv {

constexpr int kLayersPerLaunch = 64;

struct CompactLayers {
    uint4* kc[kLayersPerLaunch];
    uint4* vc[kLayersPerLaunch];
    const uint4* kt[kLayersPerLaunch];
    const uint4* vt[kLayersPerLaunch];
    int32_t num_blocks[kLayersPerLaunch];
};

// grid (B, layers); a CTA copies all accepted rows of one sequence in one layer.
// One accepted node = Hkv*D bf16 of K and of V; unit of work = one 16-byte vector.
__global__ void __launch_bounds__(256)
compact_kernel(sd_batch bt, const __grid_constant__ CompactLayers ly,
               const int32_t* __restrict__ n_acc, const int32_t* __restrict__ path,
               int32_t* status) {
    const int b = blockIdx.x;
    const int l = blockIdx.y;
    const int T = bt.T_max;
    const int na = min(n_acc[b], T);
    const int len = bt.len[b];
    const int vec_per_head = bt.D * 2 / 16;               // 16 for D = 128
    const int vec_per_node = bt.Hkv * vec_per_head;       // per K or V
    const int total = na * 2 * vec_per_node;
    for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const int k = idx / (2 * vec_per_node);
        int rem = idx - k * 2 * vec_per_node;
        const int is_v = rem / vec_per_node;
        rem -= is_v * vec_per_node;
        const int kvh = rem / vec_per_head;
        const int c = rem - kvh * vec_per_head;
        const int node = path[(size_t)b * T + k];
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

sd_status launch_compact(const sd_batch& bt, const sd_kv_layer* layers, int L,
                         const void* const* kt, const void* const* vt,
                         const int32_t* n_acc, const int32_t* path, int32_t* dev_status, cudaStream_t st) {
    for (int l0 = 0; l0 < L; l0 += kLayersPerLaunch) {
        const int nl = (L - l0 < kLayersPerLaunch) ? (L - l0) : kLayersPerLaunch;
        CompactLayers ly;
        for (int i = 0; i < nl; ++i) {
            ly.kc[i] = static_cast<uint4*>(layers[l0 + i].k);
            ly.vc[i] = static_cast<uint4*>(layers[l0 + i].v);
            ly.kt[i] = static_cast<const uint4*>(kt[l0 + i]);
            ly.vt[i] = static_cast<const uint4*>(vt[l0 + i]);
            ly.num_blocks[i] = layers[l0 + i].num_blocks;
        }
        dim3 grid(bt.B, nl);
        compact_kernel<<<grid, 256, 0, st>>>(bt, ly, n_acc, path, dev_status);
        sd_status s = cuda_ok(cudaGetLastError());
        if (s != SD_OK) return s;
    }
    return SD_OK;
}

}  // namespace sdv
