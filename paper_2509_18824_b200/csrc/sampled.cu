// Verification at a sampling temperature for deterministically drafted trees: sequential
// rejection without replacement along the tree, then one token from the residual distribution at
// the node where the walk stops.  All random numbers are inputs.
//
//   child_prob_kernel      p[b][j] = exp(logit(parent(j), token(j)) / temperature - lse(parent(j)))
//   sampled_walk_kernel    the walk: accepted path, residual mass, the stop node's drafted tokens
//   gather_stop_rows_kernel + the LM-head tcgen05 kernel in its store mode
//                          exp(logit / temperature - lse) of the stop node's row over the whole vocabulary
//   residual_blocksum_kernel  drafted tokens of the stop node zeroed, sums per 256-token block
//   residual_pick_kernel   inverse CDF in vocabulary order; writes the final token
#include "tree_device.cuh"

namespace sdv {

constexpr int kResBlock = 256;         // vocabulary tokens per CTA of residual_mass_kernel

struct SampledWs {                     // carved out of the caller's workspace
    float* p_child;                    // [B][T]
    float* resid;                      // [B]    residual mass left at the stop node
    int32_t* stop_row;                 // [B]    b * T + stop node
    int32_t* n_excl;                   // [B]
    int32_t* excl;                     // [B][64] drafted tokens of the stop node's children
    float* excl_p;                     // [B][64] and their probabilities
    float* block_sum;                  // [B][n_blocks]
    float* mass;                       // [B][V]
    uint16_t* stop_hidden;             // [B rounded up to 16][Hd] hidden rows of the stop nodes
    float* stop_lse;                   // [B]
    void* lm_ws;                       // candidate tables of the LM-head launch
};

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

size_t sampled_workspace_bytes(int B, int T, int V, int Hd) {
    const size_t nb = (size_t)(V + kResBlock - 1) / kResBlock;
    const size_t b16 = (size_t)(B + 15) / 16 * 16;
    return align256((size_t)B * T * 4) + align256((size_t)B * 4) * 3 + align256((size_t)B * 64 * 4) * 2 +
           align256((size_t)B * nb * 4) + align256((size_t)B * V * 4) + align256(b16 * Hd * 2) + align256((size_t)B * 4) +
           align256(stats_workspace_bytes(B, V));
}

static SampledWs carve(void* ws, int B, int T, int V, int Hd) {
    const size_t nb = (size_t)(V + kResBlock - 1) / kResBlock;
    char* p = static_cast<char*>(ws);
    SampledWs w;
    w.p_child = reinterpret_cast<float*>(p);   p += align256((size_t)B * T * 4);
    w.resid = reinterpret_cast<float*>(p);     p += align256((size_t)B * 4);
    w.stop_row = reinterpret_cast<int32_t*>(p); p += align256((size_t)B * 4);
    w.n_excl = reinterpret_cast<int32_t*>(p);  p += align256((size_t)B * 4);
    w.excl = reinterpret_cast<int32_t*>(p);    p += align256((size_t)B * 64 * 4);
    w.excl_p = reinterpret_cast<float*>(p);    p += align256((size_t)B * 64 * 4);
    w.block_sum = reinterpret_cast<float*>(p); p += align256((size_t)B * nb * 4);
    w.mass = reinterpret_cast<float*>(p);      p += align256((size_t)B * V * 4);
    w.stop_hidden = reinterpret_cast<uint16_t*>(p); p += align256((size_t)(B + 15) / 16 * 16 * Hd * 2);
    w.stop_lse = reinterpret_cast<float*>(p);  p += align256((size_t)B * 4);
    w.lm_ws = p;
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
                                    float* excl_p, int32_t* status) {
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
    const int tk0 = lane < n ? dt[lane] : -1, tk1 = lane + 32 < n ? dt[lane + 32] : -1;
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
            // siblings must carry distinct tokens (an earlier sibling's rejection already removed the mass)
            const int tc = dt[c];
            if (__any_sync(0xffffffffu, (pa0 == cur && lane < c && tk0 == tc) || (pa1 == cur && lane + 32 < c && tk1 == tc)))
                if (lane == 0) set_status(status, SD_ERR_INVALID_ARG);
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
    if (pa0 == cur) { excl[(size_t)b * 64 + rank0] = dt[lane]; excl_p[(size_t)b * 64 + rank0] = p_child[(size_t)b * T + lane]; }
    if (pa1 == cur) { excl[(size_t)b * 64 + rank1] = dt[lane + 32]; excl_p[(size_t)b * 64 + rank1] = p_child[(size_t)b * T + lane + 32]; }
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

// hidden rows (and their lse) of the stop nodes, gathered into a dense [B][Hd] matrix for the LM-head kernel
__global__ void gather_stop_rows_kernel(const uint16_t* __restrict__ hidden, int Hd, const float* __restrict__ lse,
                                        const int32_t* __restrict__ stop_row, uint16_t* __restrict__ stop_hidden,
                                        float* __restrict__ stop_lse) {
    const int b = blockIdx.x;
    const int row = stop_row[b];
    const uint4* src = reinterpret_cast<const uint4*>(hidden + (size_t)row * Hd);
    uint4* dst = reinterpret_cast<uint4*>(stop_hidden + (size_t)b * Hd);
    for (int i = threadIdx.x; i < Hd / 8; i += blockDim.x) dst[i] = __ldg(src + i);
    if (threadIdx.x == 0) stop_lse[b] = lse[row];
}

// grid (blocks of 256 tokens, sequences): drafted tokens of the stop node lose their mass, then the
// block's masses are summed in a fixed order (pairwise tree over the 256 positions)
__global__ void __launch_bounds__(kResBlock)
residual_blocksum_kernel(int V, const int32_t* __restrict__ n_excl, const int32_t* __restrict__ excl,
                         float* __restrict__ mass, float* __restrict__ block_sum, int n_blocks) {
    __shared__ float s_v[kResBlock];
    const int b = blockIdx.y;
    const int t = blockIdx.x * kResBlock + threadIdx.x;
    float m = 0.f;
    if (t < V) {
        m = mass[(size_t)b * V + t];
        const int ne = n_excl[b];
        bool hit = false;
        for (int e = 0; e < ne; ++e) hit |= (__ldg(excl + (size_t)b * 64 + e) == t);
        if (hit) { m = 0.f; mass[(size_t)b * V + t] = 0.f; }
    }
    s_v[threadIdx.x] = m;
    __syncthreads();
    for (int d = kResBlock / 2; d >= 1; d >>= 1) {
        if (threadIdx.x < d) s_v[threadIdx.x] += s_v[threadIdx.x + d];
        __syncthreads();
    }
    if (threadIdx.x == 0) block_sum[(size_t)b * n_blocks + blockIdx.x] = s_v[0];
}

// First index i in [0, n) at which base + v[0] + ... + v[i] reaches target, found by one warp: every
// lane sums a contiguous chunk, an inclusive scan over the lanes gives each chunk's starting value,
// and the first lane whose chunk contains the crossing walks it element by element (fixed order of
// additions).  positive_only: elements <= 0 cannot be the answer (tokens without mass).  Returns -1
// when the sum stays short; *acc_io then holds base + the whole sum; *last_pos the last index with v > 0.
__device__ __forceinline__ int warp_find_crossing(const float* v, int n, float target, bool positive_only,
                                                  float* acc_io, int* last_pos, int lane) {
    const int chunk = (n + 31) / 32;
    const int i0 = min(n, lane * chunk), i1 = min(n, i0 + chunk);
    float sum = 0.f;
    int lastp = -1;
    for (int i = i0; i < i1; ++i) { sum += v[i]; if (v[i] > 0.f) lastp = i; }
    float incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const float y = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += y;
    }
    const float before = *acc_io + (incl - sum);
    int found = -1;
    float acc_at = 0.f;
    // lanes in order: the first chunk in which the walk actually reaches the target
    uint32_t cand = __ballot_sync(0xffffffffu, i0 < i1 && before + sum >= target);
    while (cand && found < 0) {
        const int L0 = __ffs(cand) - 1;
        cand &= cand - 1;
        int idx = -1;
        float acc = before;
        if (lane == L0) {
            for (int i = i0; i < i1; ++i) {
                if (positive_only && !(v[i] > 0.f)) continue;
                if (acc + v[i] >= target) { idx = i; break; }
                acc += v[i];
            }
        }
        found = __shfl_sync(0xffffffffu, idx, L0);
        acc_at = __shfl_sync(0xffffffffu, acc, L0);
    }
    const float total = __shfl_sync(0xffffffffu, incl, 31);
    const int lp = __reduce_max_sync(0xffffffffu, lastp);
    if (last_pos && lp >= 0) *last_pos = lp;
    *acc_io = found >= 0 ? acc_at : *acc_io + total;
    return found;
}

// One CTA per sequence.  The block sums, then the masses of one block at a time, are brought into
// shared memory by all threads; warp 0 finds where the cumulative mass reaches w * (total mass).
constexpr int kPickMaxBlocks = 4096;   // vocabularies up to 1 Mi tokens
__global__ void __launch_bounds__(kResBlock)
residual_pick_kernel(sd_batch bt, int V, const float* __restrict__ w, const float* __restrict__ mass,
                     const float* __restrict__ block_sum, int n_blocks, const int32_t* __restrict__ n_acc,
                     int32_t* out_tok, int32_t* status) {
    __shared__ float s_bs[kPickMaxBlocks];
    __shared__ float s_m[kResBlock];
    __shared__ float s_acc, s_target;
    __shared__ int s_k, s_pick, s_last;
    const int b = blockIdx.x;
    const int na = n_acc[b];
    if (na < 1 || na > bt.T_max) return;                               // bad tree: already reported
    const int lane = threadIdx.x & 31;
    const float* bs = block_sum + (size_t)b * n_blocks;
    for (int k = threadIdx.x; k < n_blocks; k += blockDim.x) s_bs[k] = bs[k];
    __syncthreads();
    if (threadIdx.x < 32) {
        float total = 0.f;                                             // whole remaining mass, same order of additions
        warp_find_crossing(s_bs, n_blocks, INFINITY, false, &total, nullptr, lane);
        const float target = w[b] * total;
        float acc = 0.f;
        int k = warp_find_crossing(s_bs, n_blocks, target, false, &acc, nullptr, lane);
        if (k < 0) { k = n_blocks - 1; acc -= s_bs[k]; }               // rounding left the sum short: last block
        if (lane == 0) { s_acc = acc; s_target = target; s_k = k; s_pick = -1; s_last = -1; }
    }
    __syncthreads();
    const float* m = mass + (size_t)b * V;
    // (if the chosen block's walk stays short of the target, go on through the following blocks)
    for (int k = s_k; k < n_blocks; ++k) {
        const int t = k * kResBlock + threadIdx.x;
        s_m[threadIdx.x] = t < V ? m[t] : 0.f;
        __syncthreads();
        if (threadIdx.x < 32) {
            float acc = s_acc;
            int lastp = -1;
            const int i = warp_find_crossing(s_m, kResBlock, s_target, true, &acc, &lastp, lane);
            if (lane == 0) {
                s_acc = acc;
                if (lastp >= 0) s_last = k * kResBlock + lastp;
                if (i >= 0) s_pick = k * kResBlock + i;
            }
        }
        __syncthreads();
        if (s_pick >= 0) break;
    }
    if (threadIdx.x == 0) {
        int pick = s_pick >= 0 ? s_pick : s_last;
        if (pick < 0)                                                  // w ~ 1 and nothing left behind the chosen block:
            for (int t = V - 1; t >= 0 && pick < 0; --t)               // the last token that has mass at all
                if (m[t] > 0.f) pick = t;
        if (pick < 0) { set_status(status, SD_ERR_BOUNDS); pick = 0; }  // no mass at all: inputs were not finite
        out_tok[(size_t)b * bt.T_max + na - 1] = pick;
    }
}

// Residual draw from the LM-head pass's own statistics.  One CTA per sequence: the masses of the 32-row
// vocabulary groups of the stop row follow from (group maximum, group sum) and the row's lse; the
// drafted children's probabilities are taken out of their groups; warp 0 finds the group in which the
// cumulative mass reaches w * (total); that group's 32 logits are recomputed (32 dot products) and the
// token is found among them.  W is not streamed a second time and no logits-sized data exist.
constexpr int kPickMaxGroups = 8192;   // vocabularies up to 262144 tokens
__global__ void __launch_bounds__(256)
residual_pick_groups_kernel(sd_batch bt, const uint16_t* __restrict__ hidden, const uint16_t* __restrict__ W, int Hd, int V,
                            float inv_temp, const float* __restrict__ lse, const float2* __restrict__ group_stats, int n_groups,
                            const float* __restrict__ w, const int32_t* __restrict__ stop_row, const int32_t* __restrict__ n_excl,
                            const int32_t* __restrict__ excl, const float* __restrict__ excl_p, const int32_t* __restrict__ n_acc,
                            int32_t* out_tok, int32_t* status) {
    __shared__ float s_g[kPickMaxGroups];
    __shared__ float s_m[32];
    __shared__ float s_acc, s_target;
    __shared__ int s_k, s_pick, s_last;
    const int b = blockIdx.x;
    const int na = n_acc[b];
    if (na < 1 || na > bt.T_max) return;                               // bad tree: already reported
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = stop_row[b];
    const int M = bt.B * bt.T_max;
    const float c2 = inv_temp * 1.4426950408889634f;
    const float lse2 = lse[row] * 1.4426950408889634f;
    for (int g = threadIdx.x; g < n_groups; g += blockDim.x) {
        const float2 st = group_stats[(size_t)g * M + row];
        s_g[g] = st.y > 0.f ? st.y * exp2f(st.x * c2 - lse2) : 0.f;
    }
    __syncthreads();
    const int ne = n_excl[b];
    if (threadIdx.x == 0)                                              // drafted children carry no mass (fixed order)
        for (int e = 0; e < ne; ++e) {
            const int g = excl[(size_t)b * 64 + e] >> 5;
            s_g[g] = fmaxf(s_g[g] - excl_p[(size_t)b * 64 + e], 0.f);
        }
    __syncthreads();
    if (threadIdx.x < 32) {
        float total = 0.f;
        warp_find_crossing(s_g, n_groups, INFINITY, false, &total, nullptr, lane);
        const float target = w[b] * total;
        float acc = 0.f;
        int k = warp_find_crossing(s_g, n_groups, target, false, &acc, nullptr, lane);
        if (k < 0) { k = n_groups - 1; acc -= s_g[k]; }
        if (lane == 0) { s_acc = acc; s_target = target; s_k = k; s_pick = -1; s_last = -1; }
    }
    __syncthreads();
    const uint4* hrow = reinterpret_cast<const uint4*>(hidden + (size_t)row * Hd);
    // the 32 probabilities of group k, recomputed into s_m: eight warps, four tokens each
    auto recompute_group = [&](int k) {
        for (int i = warp * 4; i < warp * 4 + 4; ++i) {
            const int t = k * 32 + i;
            float m = 0.f;
            if (t < V) {
                const float l = warp_dot_bf16(reinterpret_cast<const uint4*>(W + (size_t)t * Hd), hrow, Hd / 8, lane);
                bool hit = false;
                for (int e = lane; e < ne; e += 32) hit |= (excl[(size_t)b * 64 + e] == t);
                m = __any_sync(0xffffffffu, hit) ? 0.f : __expf(l * inv_temp - lse[row]);
            }
            if (lane == 0) s_m[i] = m;
        }
        __syncthreads();
    };
    for (int k = s_k; k < n_groups; ++k) {
        recompute_group(k);
        if (threadIdx.x < 32) {
            float acc = s_acc;
            int lastp = -1;
            const int i = warp_find_crossing(s_m, 32, s_target, true, &acc, &lastp, lane);
            if (lane == 0) {
                s_acc = acc;
                if (lastp >= 0) s_last = k * 32 + lastp;
                if (i >= 0) s_pick = k * 32 + i;
            }
        }
        __syncthreads();
        if (s_pick >= 0) break;
    }
    // (rounding left the walk short and nothing with mass lay behind the chosen group: the last token
    //  with mass before it)
    for (int k = s_k - 1; k >= 0 && s_pick < 0 && s_last < 0; --k) {
        recompute_group(k);
        if (threadIdx.x == 0)
            for (int i = 31; i >= 0; --i)
                if (s_m[i] > 0.f) { s_last = k * 32 + i; break; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        int pick = s_pick >= 0 ? s_pick : s_last;
        if (pick < 0) { set_status(status, SD_ERR_BOUNDS); pick = 0; }  // no mass at all: inputs were not finite
        out_tok[(size_t)b * bt.T_max + na - 1] = pick;
    }
}

sd_status launch_accept_sampled(const sd_batch& bt, const void* hidden, const void* W, int Hd, int V, float inv_temp,
                                const float* lse, const float* group_stats, const int32_t* draft, const float* u, const float* w,
                                int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                                void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t st) {
    const int B = bt.B, T = bt.T_max;
    if (Hd > 16384) return SD_ERR_UNSUPPORTED;
    // vocabulary limits of the residual draw, checked before anything is launched
    if (group_stats ? ((V + 31) / 32 > kPickMaxGroups) : ((V + kResBlock - 1) / kResBlock > kPickMaxBlocks))
        return SD_ERR_UNSUPPORTED;
    if (ws_bytes < sampled_workspace_bytes(B, T, V, 16384)) return SD_ERR_WORKSPACE;
    const SampledWs s = carve(ws, B, T, V, 16384);
    const uint16_t* h = static_cast<const uint16_t*>(hidden);
    const uint16_t* Wp = static_cast<const uint16_t*>(W);
    const int n_blocks = (V + kResBlock - 1) / kResBlock;
    child_prob_kernel<<<(B * T * 32 + 127) / 128, 128, 0, st>>>(bt, h, Wp, Hd, V, inv_temp, lse, draft, s.p_child, dev_status);
    sampled_walk_kernel<<<B, 32, 0, st>>>(bt, draft, s.p_child, u, n_acc, path, out_tok, new_len, s.resid, s.stop_row,
                                         s.n_excl, s.excl, s.excl_p, dev_status);
    if (group_stats) {
        // the LM-head pass left (maximum, sum) of every 32 vocabulary rows: no second pass over W
        const int n_groups = (V + 31) / 32;
        residual_pick_groups_kernel<<<B, 256, 0, st>>>(bt, h, Wp, Hd, V, inv_temp, lse, reinterpret_cast<const float2*>(group_stats),
                                                      n_groups, w, s.stop_row, s.n_excl, s.excl, s.excl_p, n_acc, out_tok, dev_status);
        return cuda_ok(cudaGetLastError());
    }
    gather_stop_rows_kernel<<<B, 128, 0, st>>>(h, Hd, lse, s.stop_row, s.stop_hidden, s.stop_lse);
    // probabilities of the stop rows over the vocabulary: one more pass of the tensor-core LM-head kernel,
    // its epilogue storing instead of reducing (W is streamed once for all sequences)
    sd_status ls = launch_lmhead_mass(s.stop_hidden, W, B, Hd, V, inv_temp, s.stop_lse, s.mass, s.lm_ws,
                                      stats_workspace_bytes(B, V), dev_status, st);
    if (ls != SD_OK) return ls;
    residual_blocksum_kernel<<<dim3(n_blocks, B), kResBlock, 0, st>>>(V, s.n_excl, s.excl, s.mass, s.block_sum, n_blocks);
    residual_pick_kernel<<<B, kResBlock, 0, st>>>(bt, V, w, s.mass, s.block_sum, n_blocks, n_acc, out_tok, dev_status);
    return cuda_ok(cudaGetLastError());
}

}  // namespace sdv
