// KV compaction: accepted tree rows gathered into their paged cache slots,
// every layer in one launch, 16-byte vector copies.
#include "tree_device.cuh"

namespace sdv {

// grid (B, layers); a CTA copies all accepted rows of one sequence in one layer.
// One accepted node = Hkv*D bf16 of K and of V; unit of work = one 16-byte vector.
__global__ void __launch_bounds__(256)
compact_kernel(sd_batch bt, const __grid_constant__ CompactLayers ly,
               const int32_t* __restrict__ n_acc, const int32_t* __restrict__ path,
               int32_t* status) {
    const int b = blockIdx.x;
    const int na = min(n_acc[b], bt.T_max);
    compact_sequence(bt, ly, blockIdx.y, 1, b, na, path + (size_t)b * bt.T_max, threadIdx.x, blockDim.x, status);
}

void fill_compact_layers(CompactLayers* ly, const sd_kv_layer* layers, const void* const* kt, const void* const* vt,
                         int l0, int nl) {
    for (int i = 0; i < nl; ++i) {
        ly->kc[i] = static_cast<uint4*>(layers[l0 + i].k);
        ly->vc[i] = static_cast<uint4*>(layers[l0 + i].v);
        ly->kt[i] = static_cast<const uint4*>(kt[l0 + i]);
        ly->vt[i] = static_cast<const uint4*>(vt[l0 + i]);
        ly->num_blocks[i] = layers[l0 + i].num_blocks;
    }
}

sd_status launch_compact(const sd_batch& bt, const sd_kv_layer* layers, int L,
                         const void* const* kt, const void* const* vt,
                         const int32_t* n_acc, const int32_t* path, int32_t* dev_status, cudaStream_t st) {
    for (int l0 = 0; l0 < L; l0 += kLayersPerLaunch) {
        const int nl = (L - l0 < kLayersPerLaunch) ? (L - l0) : kLayersPerLaunch;
        CompactLayers ly;
        fill_compact_layers(&ly, layers, kt, vt, l0, nl);
        dim3 grid(bt.B, nl);
        compact_kernel<<<grid, 256, 0, st>>>(bt, ly, n_acc, path, dev_status);
        sd_status s = cuda_ok(cudaGetLastError());
        if (s != SD_OK) return s;
    }
    return SD_OK;
}

}  // namespace sdv
