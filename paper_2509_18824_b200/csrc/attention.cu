// Tree-masked GQA attention over a paged prefix cache plus the tree's own KV.
//
// Split-KV flash-decode: the keys of one (sequence, KV head) are cut into
// chunks; every chunk produces, for each of the T*G query rows that share this
// KV head, a partial (running max, sum of exponentials, unnormalised output);
// a merge kernel combines the partials in a fixed order.  The tree's own keys
// form one extra chunk, masked by the per-node ancestor bitmask.
#include "common.cuh"

namespace sdv {

constexpr int kRowsPerCta = 128;   // query rows (node, grouped head) per CTA
constexpr int kKeyTile = 32;       // keys staged in shared memory at a time
constexpr int kSub = 8;            // keys scored between two rescales
constexpr float kLog2e = 1.4426950408889634f;

struct AttnPlan {
    int chunk_keys;      // prefix keys per chunk (multiple of 64)
    int n_chunks;        // prefix chunks + 1 tree chunk
    int rows;            // T_max * G
    int row_blocks;
};

static AttnPlan make_plan(const sd_batch& bt) {
    AttnPlan p;
    const int G = bt.Hq / bt.Hkv;
    p.rows = bt.T_max * G;
    p.row_blocks = (p.rows + kRowsPerCta - 1) / kRowsPerCta;
    const int max_keys = bt.max_blocks_per_seq * kBlock;
    p.chunk_keys = 512;
    p.n_chunks = (max_keys + p.chunk_keys - 1) / p.chunk_keys + 1;
    return p;
}

// workspace: per (b, kvh, chunk): m[rows4], l[rows4], acc[rows][D] (fp32), rows4 = rows rounded
// up to a multiple of 4 so that every acc row stays 16-byte aligned
__host__ __device__ static inline size_t rows4(const AttnPlan& p) { return (size_t)((p.rows + 3) & ~3); }
__host__ __device__ static inline size_t partial_stride(const AttnPlan& p) { return 2 * rows4(p) + (size_t)p.rows * kD; }

size_t attention_workspace_bytes(const sd_batch& bt) {
    AttnPlan p = make_plan(bt);
    return (size_t)bt.B * bt.Hkv * p.n_chunks * partial_stride(p) * sizeof(float);
}

// One thread per query row; K/V tiles are staged in shared memory as fp32 and
// read by all threads at the same address (broadcast).
__global__ void __launch_bounds__(kRowsPerCta)
attn_partial_kernel(sd_batch bt, sd_kv_layer cache, const uint16_t* __restrict__ q,
                    const uint16_t* __restrict__ kt, const uint16_t* __restrict__ vt,
                    float scale_log2, float* __restrict__ ws, AttnPlan plan, int32_t* status) {
    __shared__ __align__(16) float Ks[kKeyTile][kD];
    __shared__ __align__(16) float Vs[kKeyTile][kD];
    extern __shared__ __align__(16) float Qs[];          // [kD][kRowsPerCta]  (transposed)

    const int chunk = blockIdx.x;
    const int rb = blockIdx.y;
    const int b = blockIdx.z / bt.Hkv;
    const int kvh = blockIdx.z % bt.Hkv;
    const int tid = threadIdx.x;
    const int G = bt.Hq / bt.Hkv;
    const int T = bt.T_max;
    const int n = min(bt.n_nodes[b], T);
    const int len = bt.len[b];
    const bool tree_chunk = (chunk == plan.n_chunks - 1);

    int key0, key1;
    if (tree_chunk) { key0 = 0; key1 = n; }
    else {
        key0 = chunk * plan.chunk_keys;
        key1 = min(len, key0 + plan.chunk_keys);
        if (key1 <= key0) return;                          // whole CTA: nothing to do
    }
    const int row = rb * kRowsPerCta + tid;
    const int node = row / G;
    const int g = row - node * G;
    const bool row_ok = (row < plan.rows) && (node < n);
    const uint64_t amask = (row_ok && tree_chunk) ? bt.anc_mask[(size_t)b * T + node] : ~0ull;

    // stage q transposed, pre-multiplied by scale * log2(e)
    {
        const uint16_t* qr = q + (((size_t)b * T + (row_ok ? node : 0)) * bt.Hq + kvh * G + (row_ok ? g : 0)) * kD;
        for (int d = 0; d < kD; d += 8) {
            uint4 u = *reinterpret_cast<const uint4*>(qr + d);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                Qs[(d + 2 * e) * kRowsPerCta + tid] = bf16lo(w[e]) * scale_log2;
                Qs[(d + 2 * e + 1) * kRowsPerCta + tid] = bf16hi(w[e]) * scale_log2;
            }
        }
    }
    float acc[kD];
#pragma unroll
    for (int d = 0; d < kD; ++d) acc[d] = 0.f;
    float m = -INFINITY, l = 0.f;

    for (int t0 = key0; t0 < key1; t0 += kKeyTile) {
        const int nk = min(kKeyTile, key1 - t0);
        __syncthreads();
        // cooperative load of nk keys: 16 vectors of 8 bf16 per row, K and V
        for (int idx = tid; idx < kKeyTile * 16; idx += kRowsPerCta) {
            const int kk = idx >> 4, c = idx & 15;
            uint4 uk = make_uint4(0, 0, 0, 0), uv = uk;
            if (kk < nk) {
                const int t = t0 + kk;
                const uint16_t *kp, *vp;
                bool ok = true;
                if (tree_chunk) {
                    const size_t off = (((size_t)b * T + t) * bt.Hkv + kvh) * kD;
                    kp = kt + off; vp = vt + off;
                } else {
                    const int blk = bt.block_table[(size_t)b * bt.max_blocks_per_seq + t / kBlock];
                    if (blk < 0 || blk >= cache.num_blocks) { set_status(status, SD_ERR_BOUNDS); ok = false; }
                    const size_t off = (((size_t)(ok ? blk : 0) * bt.Hkv + kvh) * kBlock + (t % kBlock)) * kD;
                    kp = static_cast<const uint16_t*>(cache.k) + off;
                    vp = static_cast<const uint16_t*>(cache.v) + off;
                }
                if (ok) {
                    uk = *reinterpret_cast<const uint4*>(kp + c * 8);
                    uv = *reinterpret_cast<const uint4*>(vp + c * 8);
                }
            }
            const uint32_t wk[4] = {uk.x, uk.y, uk.z, uk.w};
            const uint32_t wv[4] = {uv.x, uv.y, uv.z, uv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                Ks[kk][c * 8 + 2 * e] = bf16lo(wk[e]);
                Ks[kk][c * 8 + 2 * e + 1] = bf16hi(wk[e]);
                Vs[kk][c * 8 + 2 * e] = bf16lo(wv[e]);
                Vs[kk][c * 8 + 2 * e + 1] = bf16hi(wv[e]);
            }
        }
        __syncthreads();
        for (int s0 = 0; s0 < nk; s0 += kSub) {
            float s[kSub];
#pragma unroll
            for (int j = 0; j < kSub; ++j) s[j] = 0.f;
#pragma unroll 4
            for (int d = 0; d < kD; d += 4) {
                const float q0 = Qs[(d + 0) * kRowsPerCta + tid];
                const float q1 = Qs[(d + 1) * kRowsPerCta + tid];
                const float q2 = Qs[(d + 2) * kRowsPerCta + tid];
                const float q3 = Qs[(d + 3) * kRowsPerCta + tid];
#pragma unroll
                for (int j = 0; j < kSub; ++j) {
                    const float4 k4 = *reinterpret_cast<const float4*>(&Ks[s0 + j][d]);
                    s[j] = fmaf(q0, k4.x, s[j]);
                    s[j] = fmaf(q1, k4.y, s[j]);
                    s[j] = fmaf(q2, k4.z, s[j]);
                    s[j] = fmaf(q3, k4.w, s[j]);
                }
            }
            float mnew = m;
#pragma unroll
            for (int j = 0; j < kSub; ++j) {
                const int t = t0 + s0 + j;
                const bool vis = (s0 + j < nk) && (!tree_chunk || ((amask >> t) & 1ull));
                s[j] = vis ? s[j] : -INFINITY;
                mnew = fmaxf(mnew, s[j]);
            }
            if (mnew == -INFINITY) continue;              // nothing visible yet for this row
            const float alpha = exp2f(m - mnew);          // m = -inf gives 0
            float p[kSub];
            float psum = 0.f;
#pragma unroll
            for (int j = 0; j < kSub; ++j) { p[j] = exp2f(s[j] - mnew); psum += p[j]; }
            l = l * alpha + psum;
            m = mnew;
#pragma unroll
            for (int d = 0; d < kD; d += 4) {
                float4 o = make_float4(acc[d] * alpha, acc[d + 1] * alpha, acc[d + 2] * alpha, acc[d + 3] * alpha);
#pragma unroll
                for (int j = 0; j < kSub; ++j) {
                    const float4 v4 = *reinterpret_cast<const float4*>(&Vs[s0 + j][d]);
                    o.x = fmaf(p[j], v4.x, o.x);
                    o.y = fmaf(p[j], v4.y, o.y);
                    o.z = fmaf(p[j], v4.z, o.z);
                    o.w = fmaf(p[j], v4.w, o.w);
                }
                acc[d] = o.x; acc[d + 1] = o.y; acc[d + 2] = o.z; acc[d + 3] = o.w;
            }
        }
    }
    if (row < plan.rows) {
        float* base = ws + ((size_t)(b * bt.Hkv + kvh) * plan.n_chunks + chunk) * partial_stride(plan);
        base[row] = m;
        base[rows4(plan) + row] = l;
        float4* o = reinterpret_cast<float4*>(base + 2 * rows4(plan) + (size_t)row * kD);
#pragma unroll
        for (int d = 0; d < kD; d += 4) o[d / 4] = make_float4(acc[d], acc[d + 1], acc[d + 2], acc[d + 3]);
    }
}

// grid (T_max*G rows, Hkv, B), kD threads: thread d merges output column d.
__global__ void __launch_bounds__(kD)
attn_merge_kernel(sd_batch bt, const float* __restrict__ ws, AttnPlan plan,
                  __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    const int row = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    const int d = threadIdx.x;
    const int G = bt.Hq / bt.Hkv;
    const int T = bt.T_max;
    const int node = row / G, g = row - node * G;
    const int h = kvh * G + g;
    const size_t orow = ((size_t)b * T + node) * bt.Hq + h;
    const int n = min(bt.n_nodes[b], T);
    if (node >= n) {
        out[orow * kD + d] = __float2bfloat16(0.f);
        if (lse && d == 0) lse[orow] = 0.f;
        return;
    }
    const int len = bt.len[b];
    const float* base = ws + (size_t)(b * bt.Hkv + kvh) * plan.n_chunks * partial_stride(plan);
    float M = -INFINITY;
    for (int c = 0; c < plan.n_chunks; ++c) {
        const bool live = (c == plan.n_chunks - 1) || (c * plan.chunk_keys < len);
        if (live) M = fmaxf(M, base[(size_t)c * partial_stride(plan) + row]);
    }
    float num = 0.f, den = 0.f;
    for (int c = 0; c < plan.n_chunks; ++c) {
        const bool live = (c == plan.n_chunks - 1) || (c * plan.chunk_keys < len);
        if (!live) continue;
        const float* pc = base + (size_t)c * partial_stride(plan);
        const float w = exp2f(pc[row] - M);
        den = fmaf(w, pc[rows4(plan) + row], den);
        num = fmaf(w, pc[2 * rows4(plan) + (size_t)row * kD + d], num);
    }
    out[orow * kD + d] = __float2bfloat16(num / den);
    if (lse && d == 0) lse[orow] = (M + log2f(den)) * 0.6931471805599453f;
}

sd_status launch_attention(const sd_batch& bt, const sd_kv_layer& cache, const void* q,
                           const void* kt, const void* vt, float scale, void* out, float* lse,
                           void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t st) {
    AttnPlan plan = make_plan(bt);
    if (ws_bytes < attention_workspace_bytes(bt)) return SD_ERR_WORKSPACE;
    const size_t dyn = (size_t)kD * kRowsPerCta * sizeof(float);
    if (cudaFuncSetAttribute(attn_partial_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return SD_ERR_CUDA;
    dim3 grid(plan.n_chunks, plan.row_blocks, bt.B * bt.Hkv);
    attn_partial_kernel<<<grid, kRowsPerCta, dyn, st>>>(
        bt, cache, static_cast<const uint16_t*>(q), static_cast<const uint16_t*>(kt),
        static_cast<const uint16_t*>(vt), scale * kLog2e, static_cast<float*>(ws), plan, dev_status);
    if (cudaGetLastError() != cudaSuccess) return SD_ERR_CUDA;
    dim3 mgrid(plan.rows, bt.Hkv, bt.B);
    attn_merge_kernel<<<mgrid, kD, 0, st>>>(bt, static_cast<const float*>(ws), plan,
                                            static_cast<__nv_bfloat16*>(out), lse);
    return cuda_ok(cudaGetLastError());
}

}  // namespace sdv
