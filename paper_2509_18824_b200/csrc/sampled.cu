// Verification at a sampling temperature for deterministically drafted trees: sequential
// rejection without replacement along the tree, then one token from the residual distribution at
// the node where the walk stops.  All random numbers are inputs.
//
//   child_prob_kernel      p[b][j] = exp(logit(parent(j), token(j)) / temperature - lse(parent(j)))
//   sampled_walk_kernel    the walk: accepted path, residual mass, the stop node's drafted tokens
//   residual_mass_kernel   exp(logit / temperature - lse) of the stop node's row over the whole
//                          vocabulary (drafted tokens zeroed), per 256-token block sums
//   residual_pick_kernel   inverse CDF in vocabulary order; writes the final token
#include "tree_device.cuh"

namespace sdv {

constexpr int kResBlock = 256;         // vocabulary tokens per CTA of residual_mass_kernel
constexpr int kResMaxB = 8;            // sequences handled per launch (their hidden rows live in shared memory)

struct SampledWs {                     // carved out of the caller's workspace
    float* p_child;                    // [B][T]
    float* resid;                      // [B]    residual mass left at the stop node
    int32_t* stop_row;                 // [B]    b * T + stop node
    int32_t* n_excl;                   // [B]
    int32_t* excl;                     // [B][64] drafted tokens of the stop node's children
    float* block_sum;                  // [B][n_blocks]
    float* mass;                       // [B][V]
};

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

size_t sampled_workspace_bytes(int B, int T, int V) {
    const size_t nb = (size_t)(V + kResBlock - 1) / kResBlock;
    return align256((size_t)B * T * 4) + align256((size_t)B * 4) * 3 + align256((size_t)B * 64 * 4) +
           align256((size_t)B * nb * 4) + align256((size_t)B * V * 4);
}

static SampledWs carve(void* ws, int B, int T, int V) {
    const size_t nb = (size_t)(V + kResBlock - 1) / kResBlock;
    char* p = static_cast<char*>(ws);
    SampledWs w;
    w.p_child = reinterpret_cast<float*>(p);   p += align256((size_t)B * T * 4);
    w.resid = reinterpret_cast<float*>(p);     p += align256((size_t)B * 4);
    w.stop_row = reinterpret_cast<int32_t*>(p); p += align256((size_t)B * 4);
    w.n_excl = reinterpret_cast<int32_t*>(p);  p += align256((size_t)B * 4);
    w.excl = reinterpret_cast<int32_t*>(p);    p += align256((size_t)B * 64 * 4);
    w.block_sum = reinterpret_cast<float*>(p); p += align256((size_t)B * nb * 4);
    w.mass = reinterpret_cast<float*>(p);
    return w;
}

// dot product of two bf16 rows of length Hd (multiple of 64) by one warp, fp32, fixed order:
// lane l takes the 16-byte pieces l, l + 32, ...; lanes are combined by a butterfly
__device__ __forceinline__ float warp_dot_bf16(const uint4* __restrict__ a, const uint4* __restrict__ b, int n_vec, int lane) {
    float acc = 0.f;
    for (int i = lane; i < n_vec; i += 32) {
        const uint4 x = __ldg(a + i), y = b[i];
        acc = fmaf(bf16lo(x.x), bf16lo(y.x), acc); acc = fmaf(bf16hi(x.x), bf16hi(y.x), acc);
        acc = fmaf(bf16lo(x.y), bf16lo(y.y), acc); acc = fmaf(bf16hi(x.y), bf16hi(y.y), acc);
        acc = fmaf(bf16lo(x.z), bf16lo(y.z), acc); acc = fmaf(bf16hi(x.z), bf16hi(y.z), acc);
        acc = fmaf(bf16lo(x.w), bf16lo(y.w), acc); acc = fmaf(bf16hi(x.w), bf16hi(y.w), acc);
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
    return acc;
}

// one warp per (sequence, node >= 1)
__global__ void __launch_bounds__(128)
child_prob_kernel(sd_batch bt, const uint16_t* __restrict__ hidden, const uint16_t* __restrict__ W, int Hd, int V,
                  float inv_temp, const float* __restrict__ lse, const int32_t* __restrict__ draft,
                  float* __restrict__ p_child, int32_t* status) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int T = bt.T_max;
    if (warp >= bt.B * T) return;
    const int b = warp / T, j = warp - b * T;
    float p = 0.f;
    const int n = bt.n_nodes[b];
    if (j >= 1 && j < n && n <= T) {
        const int par = bt.parents[(size_t)b * T + j];
        const int tok = draft[(size_t)b * T + j];
        if (par < 0 || par >= j || tok < 0 || tok >= V) {
            if (lane == 0) set_status(status, par < 0 || par >= j ? SD_ERR_INVALID_TREE : SD_ERR_BOUNDS);
        } else {
            const int row = b * T + par;
            const float l = warp_dot_bf16(reinterpret_cast<const uint4*>(W + (size_t)tok * Hd),
                                          reinterpret_cast<const uint4*>(hidden + (size_t)row * Hd), Hd / 8, lane);
            p = __expf(l * inv_temp - lse[row]);
        }
    }
    if (lane == 0) p_child[(size_t)b * T + j] = p;
}

// one warp per sequence
__global__ void sampled_walk_kernel(sd_batch bt, const int32_t* __restrict__ draft, const float* __restrict__ p_child,
                                    const float* __restrict__ u, int32_t* n_acc, int32_t* path, int32_t* out_tok,
                                    int32_t* new_len, float* resid, int32_t* stop_row, int32_t* n_excl, int32_t* excl,
                                    int32_t* status) {
    const int b = blockIdx.x, lane = threadIdx.x;
    const int T = bt.T_max;
    const int n = bt.n_nodes[b];
    const int32_t* par = bt.parents + (size_t)b * T;
    const int32_t* dt = draft + (size_t)b * T;
    bool bad = (n < 1 || n > T);
    if (!bad)
        for (int i = lane; i < n; i += 32) {
            int p = par[i];
            if (i == 0 ? (p != -1) : (p < 0 || p >= i)) bad = true;
        }
    if (__any_sync(0xffffffffu, bad)) {
        if (lane == 0) { set_status(status, SD_ERR_INVALID_TREE); n_acc[b] = 0; n_excl[b] = 0; stop_row[b] = b * T; resid[b] = 0.f; }
        return;
    }
    // parent and token of the (up to) two nodes this lane looks after
    const int pa0 = lane < n ? par[lane] : -2, pa1 = lane + 32 < n ? par[lane + 32] : -2;
    int32_t* pth = path + (size_t)b * T;
    int32_t* ot = out_tok + (size_t)b * T;
    int cur = 0, na = 1;
    float R = 1.f;
    if (lane == 0) pth[0] = 0;
    while (true) {
        // children of cur, as a 64-bit mask in node order
        const uint32_t lo = __ballot_sync(0xffffffffu, pa0 == cur), hi = __ballot_sync(0xffffffffu, pa1 == cur);
        uint64_t kids = ((uint64_t)hi << 32) | lo;
        R = 1.f;
        int nxt = -1;
        while (kids) {                                       // warp-uniform loop
            const int c = __ffsll((long long)kids) - 1;
            kids &= kids - 1;
            const float pc = p_child[(size_t)b * T + c];
            if (u[(size_t)b * T + c] * R < pc) { nxt = c; break; }
            R -= pc;
        }
        if (nxt < 0) break;
        if (lane == 0) { pth[na] = nxt; ot[na - 1] = dt[nxt]; }
        cur = nxt;
        ++na;
    }
    // the stop node's drafted tokens carry no mass in the residual
    const uint32_t lo = __ballot_sync(0xffffffffu, pa0 == cur), hi = __ballot_sync(0xffffffffu, pa1 == cur);
    const int rank0 = __popc(lo & ((1u << lane) - 1u)), rank1 = __popc(lo) + __popc(hi & ((1u << lane) - 1u));
    if (pa0 == cur) excl[(size_t)b * 64 + rank0] = dt[lane];
    if (pa1 == cur) excl[(size_t)b * 64 + rank1] = dt[lane + 32];
    for (int k = na + lane; k < T; k += 32) { pth[k] = -1; ot[k] = -1; }
    if (lane == 0) {
        n_acc[b] = na;
        new_len[b] = bt.len[b] + na;
        resid[b] = R;
        stop_row[b] = b * T + cur;
        n_excl[b] = __popc(lo) + __popc(hi);
        ot[na - 1] = -1;                                     // filled by residual_pick_kernel
    }
}

// CTA = 256 consecutive vocabulary tokens, 8 warps x 32 tokens.  The stop rows of up to 8 sequences
// sit in shared memory as fp32, so every W row is read (and widened) once for all of them.  Shared
// layout of a row: the first four floats of every 8-element piece, then the second four, so that
// the lanes of a warp read consecutive 16-byte words.
__global__ void __launch_bounds__(256)
residual_mass_kernel(const uint16_t* __restrict__ hidden, const uint16_t* __restrict__ W, int Hd, int V, int b0, int nb,
                     float inv_temp, const float* __restrict__ lse, const int32_t* __restrict__ stop_row,
                     const int32_t* __restrict__ n_excl, const int32_t* __restrict__ excl,
                     float* __restrict__ mass, float* __restrict__ block_sum, int n_blocks) {
    extern __shared__ __align__(16) uint8_t rsm[];
    const int n_vec = Hd / 8;
    float4* rows = reinterpret_cast<float4*>(rsm);                          // [nb][2][n_vec]
    float* vals = reinterpret_cast<float*>(rsm + (size_t)nb * Hd * 4);      // [nb][256]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < nb * n_vec; i += blockDim.x) {
        const int b = i / n_vec, k = i - b * n_vec;
        const uint4 x = __ldg(reinterpret_cast<const uint4*>(hidden + (size_t)stop_row[b0 + b] * Hd) + k);
        rows[(size_t)(b * 2) * n_vec + k] = make_float4(bf16lo(x.x), bf16hi(x.x), bf16lo(x.y), bf16hi(x.y));
        rows[(size_t)(b * 2 + 1) * n_vec + k] = make_float4(bf16lo(x.z), bf16hi(x.z), bf16lo(x.w), bf16hi(x.w));
    }
    __syncthreads();
    for (int k = 0; k < 32; ++k) {
        const int t_in = warp * 32 + k;
        const int t = blockIdx.x * kResBlock + t_in;
        float acc[kResMaxB];
#pragma unroll
        for (int b = 0; b < kResMaxB; ++b) acc[b] = 0.f;
        if (t < V) {
            const uint4* wrow = reinterpret_cast<const uint4*>(W + (size_t)t * Hd);
            for (int i = lane; i < n_vec; i += 32) {
                const uint4 x = __ldg(wrow + i);
                const float w0 = bf16lo(x.x), w1 = bf16hi(x.x), w2 = bf16lo(x.y), w3 = bf16hi(x.y);
                const float w4 = bf16lo(x.z), w5 = bf16hi(x.z), w6 = bf16lo(x.w), w7 = bf16hi(x.w);
#pragma unroll
                for (int b = 0; b < kResMaxB; ++b) {
                    if (b < nb) {
                        const float4 y0 = rows[(size_t)(b * 2) * n_vec + i], y1 = rows[(size_t)(b * 2 + 1) * n_vec + i];
                        float a = acc[b];
                        a = fmaf(w0, y0.x, a); a = fmaf(w1, y0.y, a); a = fmaf(w2, y0.z, a); a = fmaf(w3, y0.w, a);
                        a = fmaf(w4, y1.x, a); a = fmaf(w5, y1.y, a); a = fmaf(w6, y1.z, a); a = fmaf(w7, y1.w, a);
                        acc[b] = a;
                    }
                }
            }
        }
#pragma unroll
        for (int b = 0; b < kResMaxB; ++b) {
            if (b < nb) {
                float l = acc[b];
#pragma unroll
                for (int d = 16; d >= 1; d >>= 1) l += __shfl_xor_sync(0xffffffffu, l, d);
                float m = 0.f;
                if (t < V) {
                    const int ne = n_excl[b0 + b];                     // drafted tokens of the stop node carry no mass
                    bool hit = false;
                    for (int e = lane; e < ne; e += 32) hit |= (excl[(size_t)(b0 + b) * 64 + e] == t);
                    m = __any_sync(0xffffffffu, hit) ? 0.f : __expf(l * inv_temp - lse[stop_row[b0 + b]]);
                }
                if (lane == 0) {
                    vals[b * kResBlock + t_in] = m;
                    if (t < V) mass[(size_t)(b0 + b) * V + t] = m;
                }
            }
        }
    }
    __syncthreads();
    if (threadIdx.x < nb) {                                            // block sums in vocabulary order
        float s = 0.f;
        for (int i = 0; i < kResBlock; ++i) s += vals[threadIdx.x * kResBlock + i];
        block_sum[(size_t)(b0 + threadIdx.x) * n_blocks + blockIdx.x] = s;
    }
}

// one thread per sequence walks the block sums, then the block's tokens, in vocabulary order
__global__ void residual_pick_kernel(sd_batch bt, int V, const float* __restrict__ w, const float* __restrict__ mass,
                                     const float* __restrict__ block_sum, int n_blocks, const int32_t* __restrict__ n_acc,
                                     int32_t* out_tok, int32_t* status) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= bt.B) return;
    const int na = n_acc[b];
    if (na < 1 || na > bt.T_max) return;                               // bad tree: already reported
    const float* bs = block_sum + (size_t)b * n_blocks;
    float total = 0.f;
    for (int k = 0; k < n_blocks; ++k) total += bs[k];
    const float target = w[b] * total;
    float acc = 0.f;
    int k = 0;
    for (; k < n_blocks - 1; ++k) {
        if (acc + bs[k] >= target) break;
        acc += bs[k];
    }
    const float* m = mass + (size_t)b * V;
    int pick = -1, last = -1;
    // (if rounding leaves the sums short, fall through the following blocks to the last token with mass)
    for (; k < n_blocks && pick < 0; ++k) {
        const int t1 = min(V, (k + 1) * kResBlock);
        for (int t = k * kResBlock; t < t1; ++t) {
            const float mt = m[t];
            if (mt <= 0.f) continue;
            last = t;
            if (acc + mt >= target) { pick = t; break; }
            acc += mt;
        }
    }
    if (pick < 0) pick = last;
    if (pick < 0) { set_status(status, SD_ERR_BOUNDS); pick = 0; }      // no mass at all: inputs were not finite
    out_tok[(size_t)b * bt.T_max + na - 1] = pick;
}

sd_status launch_accept_sampled(const sd_batch& bt, const void* hidden, const void* W, int Hd, int V, float inv_temp,
                                const float* lse, const int32_t* draft, const float* u, const float* w,
                                int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                                void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t st) {
    const int B = bt.B, T = bt.T_max;
    if (ws_bytes < sampled_workspace_bytes(B, T, V)) return SD_ERR_WORKSPACE;
    const SampledWs s = carve(ws, B, T, V);
    const uint16_t* h = static_cast<const uint16_t*>(hidden);
    const uint16_t* Wp = static_cast<const uint16_t*>(W);
    const int n_blocks = (V + kResBlock - 1) / kResBlock;
    child_prob_kernel<<<(B * T * 32 + 127) / 128, 128, 0, st>>>(bt, h, Wp, Hd, V, inv_temp, lse, draft, s.p_child, dev_status);
    sampled_walk_kernel<<<B, 32, 0, st>>>(bt, draft, s.p_child, u, n_acc, path, out_tok, new_len, s.resid, s.stop_row,
                                         s.n_excl, s.excl, dev_status);
    for (int b0 = 0; b0 < B; b0 += kResMaxB) {
        const int nb = (B - b0 < kResMaxB) ? (B - b0) : kResMaxB;
        const size_t smem = (size_t)nb * Hd * 4 + (size_t)nb * kResBlock * 4;
        if (smem > 200 * 1024) return SD_ERR_UNSUPPORTED;
        if (cudaFuncSetAttribute(residual_mass_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return SD_ERR_CUDA;
        residual_mass_kernel<<<n_blocks, 256, smem, st>>>(h, Wp, Hd, V, b0, nb, inv_temp, lse, s.stop_row, s.n_excl, s.excl,
                                                         s.mass, s.block_sum, n_blocks);
    }
    residual_pick_kernel<<<(B + 31) / 32, 32, 0, st>>>(bt, V, w, s.mass, s.block_sum, n_blocks, n_acc, out_tok, dev_status);
    return cuda_ok(cudaGetLastError());
}

}  // namespace sdv
