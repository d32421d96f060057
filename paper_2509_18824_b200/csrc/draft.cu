// Draft-side target-feature aggregation (Sec. 3.1.1 of the paper): Q meta queries, shared by all
// tokens, attend over the L target-layer features of each token; the core of that cross-attention
// for head size 128.  Streaming work: every token's K and V rows (L x D each) are read once, so the
// roofline is HBM bandwidth.  One warp per (token, head).  The two tiny products (Q x 128 x L and
// Q x L x 128, Q <= 8) run as warp-level mma.sync m16n8k16 (rows 8..15 of the A operands are zero):
// with scalar FMAs the kernel was instruction-bound at a third of the memory bandwidth, and a
// tcgen05 tile (M = 128, TMEM, one issuing thread per CTA) has no use for 4 query rows per token.
#include "common.cuh"

namespace sdv {

constexpr int kDh = 128;               // head size
constexpr int kDraftWarps = 4;         // 128 threads, three CTAs per SM
constexpr int kVRow = kDh * 2 + 16;    // bytes per staged V row: 16 bytes of padding keep ldmatrix conflict-free
constexpr int kVTile = 32 * kVRow;     // one warp's V tile (32 layers)

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// SAME: k and v are one buffer (the un-projected reading); every row is then fetched once, into the
// shared tile, and the K fragments come from that tile too (plain ldmatrix) instead of from global memory.
template <bool SAME>
__global__ void __launch_bounds__(kDraftWarps * 32, 3)
draft_feature_attention_kernel(const uint16_t* __restrict__ qp, const uint16_t* __restrict__ k,
                               const uint16_t* __restrict__ v, int S, int L, int Q, int H, float scale,
                               uint16_t* __restrict__ out) {
    extern __shared__ __align__(16) uint8_t dsm[];
    const int D = H * kDh;
    uint16_t* qs = reinterpret_cast<uint16_t*>(dsm);                                // [Q][D] meta queries
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t* vs = dsm + (((size_t)Q * D * 2 + 15) & ~(size_t)15) + (size_t)warp * kVTile;   // this warp's V tile
    for (int i = threadIdx.x; i < Q * D / 8; i += blockDim.x)
        reinterpret_cast<uint4*>(qs)[i] = __ldg(reinterpret_cast<const uint4*>(qp) + i);
    for (int i = lane; i < kVTile / 16; i += 32)                                    // rows >= L stay zero
        reinterpret_cast<uint4*>(vs)[i] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    const int g = lane >> 2, t = lane & 3;                                          // mma fragment coordinates
    const uint32_t vs_addr = (uint32_t)__cvta_generic_to_shared(vs);
    const float scale_log2 = scale * 1.4426950408889634f;
    const long long tasks = (long long)S * H;
    for (long long task = (long long)blockIdx.x * kDraftWarps + warp; task < tasks; task += (long long)gridDim.x * kDraftWarps) {
        const int s = (int)(task / H), h = (int)(task - (long long)s * H);
        const uint16_t* kh = k + ((size_t)s * L) * D + (size_t)h * kDh;
        const uint16_t* vh = v + ((size_t)s * L) * D + (size_t)h * kDh;
        // ---- V rows of this head into shared memory (asynchronous copies, 16 bytes each, coalesced)
        for (int idx = lane; idx < L * (kDh / 8); idx += 32) {
            const int row = idx >> 4, c16 = idx & 15;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                         ::"r"(vs_addr + row * kVRow + c16 * 16), "l"(vh + (size_t)row * D + c16 * 8) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        // ---- K rows as B fragments (layer 8 * nt + g, values 16 * ks + 2t .. and + 8)
        uint32_t kb[4][8][2];
        if (SAME) {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncwarp();
            const int mi_ = lane >> 3, r_ = lane & 7;
#pragma unroll
            for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                for (int kp = 0; kp < 4; ++kp)                                      // two k-steps per load
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(kb[nt][2 * kp][0]), "=r"(kb[nt][2 * kp][1]), "=r"(kb[nt][2 * kp + 1][0]), "=r"(kb[nt][2 * kp + 1][1])
                                 : "r"(vs_addr + (nt * 8 + r_) * kVRow + (2 * kp + (mi_ >> 1)) * 32 + (mi_ & 1) * 16) : "memory");
        } else {                                                                    // 4-byte loads, all in flight
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const int row = nt * 8 + g;
                const uint32_t* kr = reinterpret_cast<const uint32_t*>(kh + (size_t)min(row, L - 1) * D) + t;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    kb[nt][ks][0] = __ldg(kr + ks * 8);
                    kb[nt][ks][1] = __ldg(kr + ks * 8 + 4);
                }
            }
        }
        // ---- meta queries of this head as A fragments (row g; rows >= Q and rows 8..15 are zero)
        uint32_t qa[8][2];
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint32_t* qr = reinterpret_cast<const uint32_t*>(qs + (size_t)min(g, Q - 1) * D + h * kDh) + t;
            qa[ks][0] = g < Q ? qr[ks * 8] : 0u;
            qa[ks][1] = g < Q ? qr[ks * 8 + 4] : 0u;
        }
        // ---- scores S[q][l]
        float sc[4][4];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) mma_bf16_16816(sc[nt], qa[ks][0], 0u, qa[ks][1], 0u, kb[nt][ks][0], kb[nt][ks][1]);
        }
        // ---- soft-max over the layers: row g lives in the four lanes with this g, columns 8 nt + 2t, + 1
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const int l0 = nt * 8 + 2 * t;
            sc[nt][0] = l0 < L ? sc[nt][0] * scale_log2 : -INFINITY;
            sc[nt][1] = l0 + 1 < L ? sc[nt][1] * scale_log2 : -INFINITY;
            mx = fmaxf(mx, fmaxf(sc[nt][0], sc[nt][1]));
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        float sum = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            sc[nt][0] = exp2f(sc[nt][0] - mx); sc[nt][1] = exp2f(sc[nt][1] - mx);
            sum += sc[nt][0] + sc[nt][1];
        }
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        const float inv = 1.f / sum;
        // probabilities as A fragments of the second product (k = layer): tiles 2 ks and 2 ks + 1
        uint32_t pa[2][2];
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
            pa[ks][0] = pack_bf16(sc[2 * ks][0] * inv, sc[2 * ks][1] * inv);
            pa[ks][1] = pack_bf16(sc[2 * ks + 1][0] * inv, sc[2 * ks + 1][1] * inv);
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();
        // ---- out[q][d] = sum_l P[q][l] V[l][d]; V fragments by transposing loads from shared memory
        const int mi = lane >> 3, r = lane & 7;
        const uint32_t lm_base = vs_addr + ((mi & 1) * 8 + r) * kVRow + (mi >> 1) * 16;
        uint16_t* orow = out + ((size_t)s * Q + min(g, Q - 1)) * D + (size_t)h * kDh + 2 * t;
#pragma unroll
        for (int np = 0; np < 8; ++np) {                                             // 16 output values per step
            float o0[4] = {0.f, 0.f, 0.f, 0.f}, o1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                uint32_t b0, b1, b2, b3;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(b0), "=r"(b1), "=r"(b2), "=r"(b3)
                             : "r"(lm_base + ks * 16 * kVRow + np * 32) : "memory");
                mma_bf16_16816(o0, pa[ks][0], 0u, pa[ks][1], 0u, b0, b1);
                mma_bf16_16816(o1, pa[ks][0], 0u, pa[ks][1], 0u, b2, b3);
            }
            if (g < Q) {
                *reinterpret_cast<uint32_t*>(orow + np * 16) = pack_bf16(o0[0], o0[1]);
                *reinterpret_cast<uint32_t*>(orow + np * 16 + 8) = pack_bf16(o1[0], o1[1]);
            }
        }
        __syncwarp();                                                                // the V tile is refilled by the next task
    }
}

sd_status launch_draft_feature_attention(const void* qp, const void* k, const void* v, int S, int L, int Q, int H,
                                         float scale, void* out, cudaStream_t st) {
    const int D = H * kDh;
    const size_t smem = (((size_t)Q * D * 2 + 15) & ~(size_t)15) + (size_t)kDraftWarps * kVTile;
    if (smem > 200 * 1024) return SD_ERR_UNSUPPORTED;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return SD_ERR_CUDA;
    const long long tasks = (long long)S * H;
    const long long want = (tasks + kDraftWarps - 1) / kDraftWarps;
    const long long cap = (long long)sms * 6;                        // resident CTAs, grid-stride beyond
    const int grid = (int)(want < cap ? want : cap);
    auto kern = (k == v) ? draft_feature_attention_kernel<true> : draft_feature_attention_kernel<false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SD_ERR_CUDA;
    kern<<<grid, kDraftWarps * 32, smem, st>>>(
        static_cast<const uint16_t*>(qp), static_cast<const uint16_t*>(k), static_cast<const uint16_t*>(v), S, L, Q, H, scale,
        static_cast<uint16_t*>(out));
    return cuda_ok(cudaGetLastError());
}

}  // namespace sdv
