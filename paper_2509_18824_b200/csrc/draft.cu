// Draft-side target-feature aggregation (Sec. 3.1.1 of the paper): Q meta queries, shared by all
// tokens, attend over the L target-layer features of each token; the core of that cross-attention
// for head size 128.  Pure streaming work: every token's K and V rows (L x D each) are read once,
// so the roofline is HBM bandwidth; one warp per (token, head), no tensor cores (Q is 1..8 rows).
#include "common.cuh"

namespace sdv {

constexpr int kDh = 128;               // head size
constexpr int kDraftWarps = 8;

// QP = Q rounded up to 1, 2, 4 or 8 (register accumulators); rows >= Q are skipped by predicate.
template <int QP>
__global__ void __launch_bounds__(kDraftWarps * 32)
draft_feature_attention_kernel(const uint16_t* __restrict__ qp, const uint16_t* __restrict__ k,
                               const uint16_t* __restrict__ v, int S, int L, int Q, int H, float scale,
                               uint16_t* __restrict__ out) {
    extern __shared__ __align__(16) uint8_t dsm[];
    const int D = H * kDh;
    float* qs = reinterpret_cast<float*>(dsm);                       // [Q][D] meta queries, fp32
    float* ps = qs + (size_t)Q * D;                                  // [warps][QP][32] probabilities
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < Q * D / 2; i += blockDim.x) {
        const uint32_t x = __ldg(reinterpret_cast<const uint32_t*>(qp) + i);
        qs[2 * i] = bf16lo(x); qs[2 * i + 1] = bf16hi(x);
    }
    __syncthreads();
    float* pw = ps + (size_t)warp * QP * 32;
    const long long tasks = (long long)S * H;
    for (long long task = (long long)blockIdx.x * kDraftWarps + warp; task < tasks; task += (long long)gridDim.x * kDraftWarps) {
        const int s = (int)(task / H), h = (int)(task - (long long)s * H);
        // ---- scores: lane l owns layer l; its K row of this head is 256 contiguous bytes
        float acc[QP];
#pragma unroll
        for (int q = 0; q < QP; ++q) acc[q] = 0.f;
        if (lane < L) {
            const uint4* krow = reinterpret_cast<const uint4*>(k + ((size_t)s * L + lane) * D + (size_t)h * kDh);
#pragma unroll
            for (int c = 0; c < kDh / 8; ++c) {
                const uint4 x = __ldg(krow + c);
                const float x0 = bf16lo(x.x), x1 = bf16hi(x.x), x2 = bf16lo(x.y), x3 = bf16hi(x.y);
                const float x4 = bf16lo(x.z), x5 = bf16hi(x.z), x6 = bf16lo(x.w), x7 = bf16hi(x.w);
#pragma unroll
                for (int q = 0; q < QP; ++q) {
                    if (q < Q) {
                        const float4 a = *reinterpret_cast<const float4*>(qs + (size_t)q * D + h * kDh + c * 8);
                        const float4 b = *reinterpret_cast<const float4*>(qs + (size_t)q * D + h * kDh + c * 8 + 4);
                        float t = acc[q];
                        t = fmaf(x0, a.x, t); t = fmaf(x1, a.y, t); t = fmaf(x2, a.z, t); t = fmaf(x3, a.w, t);
                        t = fmaf(x4, b.x, t); t = fmaf(x5, b.y, t); t = fmaf(x6, b.z, t); t = fmaf(x7, b.w, t);
                        acc[q] = t;
                    }
                }
            }
        }
        // ---- soft-max over the layers (= over the lanes), per query
#pragma unroll
        for (int q = 0; q < QP; ++q) {
            if (q < Q) {
                const float sc = lane < L ? acc[q] * scale : -INFINITY;
                float m = sc;
#pragma unroll
                for (int d = 16; d >= 1; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
                const float e = lane < L ? __expf(sc - m) : 0.f;
                float sum = e;
#pragma unroll
                for (int d = 16; d >= 1; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
                pw[q * 32 + lane] = e / sum;
            }
        }
        __syncwarp();
        // ---- out = P . V: lane owns 4 of the head's 128 values; a V row is 256 coalesced bytes
        float o[QP][4];
#pragma unroll
        for (int q = 0; q < QP; ++q) { o[q][0] = o[q][1] = o[q][2] = o[q][3] = 0.f; }
        const uint2* vbase = reinterpret_cast<const uint2*>(v + ((size_t)s * L) * D + (size_t)h * kDh) + lane;
        for (int l = 0; l < L; ++l) {
            const uint2 x = __ldg(vbase + (size_t)l * (D / 4));
            const float v0 = bf16lo(x.x), v1 = bf16hi(x.x), v2 = bf16lo(x.y), v3 = bf16hi(x.y);
#pragma unroll
            for (int q = 0; q < QP; ++q) {
                if (q < Q) {
                    const float p = pw[q * 32 + l];
                    o[q][0] = fmaf(p, v0, o[q][0]); o[q][1] = fmaf(p, v1, o[q][1]);
                    o[q][2] = fmaf(p, v2, o[q][2]); o[q][3] = fmaf(p, v3, o[q][3]);
                }
            }
        }
#pragma unroll
        for (int q = 0; q < QP; ++q) {
            if (q < Q) {
                __nv_bfloat162 a = __floats2bfloat162_rn(o[q][0], o[q][1]), b = __floats2bfloat162_rn(o[q][2], o[q][3]);
                uint2 w;
                w.x = *reinterpret_cast<uint32_t*>(&a); w.y = *reinterpret_cast<uint32_t*>(&b);
                reinterpret_cast<uint2*>(out + ((size_t)s * Q + q) * D + (size_t)h * kDh)[lane] = w;
            }
        }
        __syncwarp();                                                // pw is rewritten by the next task
    }
}

sd_status launch_draft_feature_attention(const void* qp, const void* k, const void* v, int S, int L, int Q, int H,
                                         float scale, void* out, cudaStream_t st) {
    const int D = H * kDh;
    const int QP = Q <= 1 ? 1 : Q <= 2 ? 2 : Q <= 4 ? 4 : 8;
    const size_t smem = (size_t)Q * D * 4 + (size_t)kDraftWarps * QP * 32 * 4;
    if (smem > 200 * 1024) return SD_ERR_UNSUPPORTED;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return SD_ERR_CUDA;
    const long long tasks = (long long)S * H;
    long long want = (tasks + kDraftWarps - 1) / kDraftWarps;
    const long long cap = (long long)sms * 4;                        // a few resident CTAs per SM, grid-stride beyond
    const int grid = (int)(want < cap ? want : cap);
    auto go = [&](auto kern) -> sd_status {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return SD_ERR_CUDA;
        kern<<<grid, kDraftWarps * 32, smem, st>>>(static_cast<const uint16_t*>(qp), static_cast<const uint16_t*>(k),
                                                    static_cast<const uint16_t*>(v), S, L, Q, H, scale,
                                                    static_cast<uint16_t*>(out));
        return cuda_ok(cudaGetLastError());
    };
    switch (QP) {
        case 1: return go(draft_feature_attention_kernel<1>);
        case 2: return go(draft_feature_attention_kernel<2>);
        case 4: return go(draft_feature_attention_kernel<4>);
        default: return go(draft_feature_attention_kernel<8>);
    }
}

}  // namespace sdv
