// LM-head projection with fused arg-max: logits never reach memory.
// Each CTA computes a (rows x vocab) tile of hidden . W^T, keeps only the
// per-row (max, lowest index) of its vocabulary slab, and a second kernel
// reduces the slabs.
#include "common.cuh"

namespace sdv {

constexpr int kTM = 64;     // rows per CTA
constexpr int kTN = 128;    // vocabulary entries per CTA
constexpr int kTK = 32;     // contraction step

size_t lmhead_workspace_bytes(int M, int V) {
    const size_t slabs = (size_t)(V + kTN - 1) / kTN;
    return (size_t)M * slabs * (sizeof(float) + sizeof(int32_t));
}

__device__ __forceinline__ void better(float& v, int& i, float v2, int i2) {
    if (v2 > v || (v2 == v && i2 < i)) { v = v2; i = i2; }
}

__global__ void __launch_bounds__(256)
lmhead_tile_kernel(const uint16_t* __restrict__ hidden, const uint16_t* __restrict__ W,
                   int M, int Hd, int V, int slabs, float* __restrict__ pmax, int32_t* __restrict__ pidx) {
    __shared__ __align__(16) float As[kTK][kTM + 4];
    __shared__ __align__(16) float Bs[kTK][kTN + 4];
    const int tid = threadIdx.x;
    const int r0 = blockIdx.x * kTM;
    const int v0 = blockIdx.y * kTN;
    const int ty = tid >> 4, tx = tid & 15;       // 16 x 16 threads: 4 rows x 8 vocab entries each
    float acc[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < Hd; k0 += kTK) {
        {   // A tile: 64 rows x 32 k = 256 vectors of 8
            const int r = tid >> 2, c = tid & 3;
            uint4 u = make_uint4(0, 0, 0, 0);
            if (r0 + r < M) u = *reinterpret_cast<const uint4*>(hidden + (size_t)(r0 + r) * Hd + k0 + c * 8);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                As[c * 8 + 2 * e][r] = bf16lo(w[e]);
                As[c * 8 + 2 * e + 1][r] = bf16hi(w[e]);
            }
        }
#pragma unroll
        for (int it = 0; it < 2; ++it) {   // B tile: 128 vocab x 32 k = 512 vectors
            const int idx = tid + it * 256;
            const int r = idx >> 2, c = idx & 3;
            uint4 u = make_uint4(0, 0, 0, 0);
            if (v0 + r < V) u = *reinterpret_cast<const uint4*>(W + (size_t)(v0 + r) * Hd + k0 + c * 8);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                Bs[c * 8 + 2 * e][r] = bf16lo(w[e]);
                Bs[c * 8 + 2 * e + 1][r] = bf16hi(w[e]);
            }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kTK; ++k) {
            const float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 8]);
            const float4 b1 = *reinterpret_cast<const float4*>(&Bs[k][tx * 8 + 4]);
            const float av[4] = {a.x, a.y, a.z, a.w};
            const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float bv = -INFINITY;
        int bi = 0x7fffffff;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int v = v0 + tx * 8 + j;
            if (v < V) better(bv, bi, acc[i][j], v);
        }
#pragma unroll
        for (int off = 8; off >= 1; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
            better(bv, bi, ov, oi);
        }
        const int r = r0 + ty * 4 + i;
        if (tx == 0 && r < M) {
            pmax[(size_t)r * slabs + blockIdx.y] = bv;
            pidx[(size_t)r * slabs + blockIdx.y] = bi;
        }
    }
}

// one warp per row
__global__ void lmhead_reduce_kernel(const float* __restrict__ pmax, const int32_t* __restrict__ pidx,
                                     int M, int slabs, int32_t* __restrict__ argmax, float* __restrict__ maxlogit) {
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= M) return;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int s = lane; s < slabs; s += 32) better(bv, bi, pmax[(size_t)r * slabs + s], pidx[(size_t)r * slabs + s]);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
        better(bv, bi, ov, oi);
    }
    if (lane == 0) {
        argmax[r] = bi;
        if (maxlogit) maxlogit[r] = bv;
    }
}

sd_status launch_lmhead(const void* hidden, const void* W, int M, int Hd, int V,
                        int32_t* argmax, float* maxlogit, void* ws, size_t ws_bytes,
                        int32_t* dev_status, cudaStream_t st) {
    (void)dev_status;
    if (ws_bytes < lmhead_workspace_bytes(M, V)) return SD_ERR_WORKSPACE;
    const int slabs = (V + kTN - 1) / kTN;
    float* pmax = static_cast<float*>(ws);
    int32_t* pidx = reinterpret_cast<int32_t*>(pmax + (size_t)M * slabs);
    dim3 grid((M + kTM - 1) / kTM, slabs);
    lmhead_tile_kernel<<<grid, 256, 0, st>>>(static_cast<const uint16_t*>(hidden), static_cast<const uint16_t*>(W),
                                             M, Hd, V, slabs, pmax, pidx);
    if (cudaGetLastError() != cudaSuccess) return SD_ERR_CUDA;
    lmhead_reduce_kernel<<<(M + 3) / 4, 128, 0, st>>>(pmax, pidx, M, slabs, argmax, maxlogit);
    return cuda_ok(cudaGetLastError());
}

}  // namespace sdv
