// Verification at a sampling temperature for deterministically drafted trees: sequential
// rejection without replacement along the tree, then one token from the residual distribution at
// the node where the walk stops.  All random numbers are inputs.
//
// The steps are device functions, used by the stand-alone kernels behind sd_accept_tree_sampled and by
// the one tail kernel behind sd_lmhead_accept_sampled_compact:
//   child_prob             p[b][j] = exp(logit(parent(j), token(j)) / temperature - lse(parent(j)))
//   sampled_walk           the walk: accepted path, residual mass, the stop node's drafted tokens
//   residual_pick_groups   the last token from the LM-head pass's per-group (maximum, sum) table
// Without that table the stand-alone call goes over W a second time:
//   gather_stop_rows_kernel + the LM-head tcgen05 kernel in its store mode
//                          exp(logit / temperature - lse) of the stop node's row over the whole vocabulary
//   residual_blocksum_kernel  drafted tokens of the stop node zeroed, sums per 256-token block
//   residual_pick_kernel   inverse CDF in vocabulary order; writes the final token
#include "tree_device.cuh"
#include "sm100.cuh"

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

__device__ __forceinline__ float fma8_bf16(const uint4& x, const uint4& y, float acc) {
    acc = fmaf(bf16lo(x.x), bf16lo(y.x), acc); acc = fmaf(bf16hi(x.x), bf16hi(y.x), acc);
    acc = fmaf(bf16lo(x.y), bf16lo(y.y), acc); acc = fmaf(bf16hi(x.y), bf16hi(y.y), acc);
    acc = fmaf(bf16lo(x.z), bf16lo(y.z), acc); acc = fmaf(bf16hi(x.z), bf16hi(y.z), acc);
    acc = fmaf(bf16lo(x.w), bf16lo(y.w), acc); acc = fmaf(bf16hi(x.w), bf16hi(y.w), acc);
    return acc;
}

// Dot products of NR bf16 rows a[0..NR) with one bf16 row b, all of length 8 * n_vec (Hd, a multiple of
// 64), by one warp, fp32, fixed order: lane l takes the 16-byte pieces l, l + 32, ... in that order;
// lanes are combined by a butterfly.  The loads of a batch of pieces are issued before its arithmetic
// (latency-bound: every load in flight at once), which does not change the order of the additions.
template <int NR>
__device__ __forceinline__ void warp_dots_bf16(const uint4* (&a)[NR], const uint4* b, int n_vec, int lane, float (&out)[NR]) {
    constexpr int kAhead = NR >= 4 ? 4 : 8;            // pieces per lane in flight, per row (more did not help: one SM's load path is the limit)
    float acc[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) acc[r] = 0.f;
    for (int i0 = lane; i0 < n_vec; i0 += 32 * kAhead) {
        uint4 x[NR][kAhead], y[kAhead];
#pragma unroll
        for (int k = 0; k < kAhead; ++k) {
            const int i = i0 + 32 * k;
            if (i < n_vec) {
                y[k] = b[i];
#pragma unroll
                for (int r = 0; r < NR; ++r) x[r][k] = __ldg(a[r] + i);
            }
        }
#pragma unroll
        for (int k = 0; k < kAhead; ++k)
            if (i0 + 32 * k < n_vec) {
#pragma unroll
                for (int r = 0; r < NR; ++r) acc[r] = fma8_bf16(x[r][k], y[k], acc[r]);
            }
    }
#pragma unroll
    for (int r = 0; r < NR; ++r) {
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], d);
        out[r] = acc[r];
    }
}

// Probability, under its parent's target distribution, of the token drafted at node j of sequence b
// (0 for the root and for unused nodes); one warp.  lse: log sum exp of the LM-head rows.
__device__ __forceinline__ float child_prob(const sd_batch& bt, int b, int j, int lane, const uint16_t* __restrict__ hidden,
                                            const uint16_t* __restrict__ W, int Hd, int V, float inv_temp, const float* lse,
                                            const int32_t* __restrict__ draft, int32_t* status) {
    const int T = bt.T_max;
    const int n = bt.n_nodes[b];
    if (!(j >= 1 && j < n && n <= T)) return 0.f;
    const int par = bt.parents[(size_t)b * T + j];
    const int tok = draft[(size_t)b * T + j];
    if (par < 0 || par >= j || tok < 0 || tok >= V) {
        if (lane == 0) set_status(status, par < 0 || par >= j ? SD_ERR_INVALID_TREE : SD_ERR_BOUNDS);
        return 0.f;
    }
    const int row = b * T + par;
    const uint4* wrow[1] = {reinterpret_cast<const uint4*>(W + (size_t)tok * Hd)};
    float l[1];
    warp_dots_bf16<1>(wrow, reinterpret_cast<const uint4*>(hidden + (size_t)row * Hd), Hd / 8, lane, l);
    return __expf(l[0] * inv_temp - lse[row]);
}

// one warp per (sequence, node)
__global__ void __launch_bounds__(128)
child_prob_kernel(sd_batch bt, const uint16_t* __restrict__ hidden, const uint16_t* __restrict__ W, int Hd, int V,
                  float inv_temp, const float* __restrict__ lse, const int32_t* __restrict__ draft,
                  float* __restrict__ p_child, int32_t* status) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int T = bt.T_max;
    if (warp >= bt.B * T) return;
    const int b = warp / T, j = warp - b * T;
    const float p = child_prob(bt, b, j, lane, hidden, W, Hd, V, inv_temp, lse, draft, status);
    if (lane == 0) p_child[(size_t)b * T + j] = p;
}

// The rejection walk of one sequence, by one warp.  Results go where `o` points (global or shared
// memory): the accepted path and the drafted tokens along it (entries beyond: -1; the slot of the
// token still to be drawn: -1), the drafted tokens of the stop node's children and their
// probabilities.  Returns, in every lane: accepted nodes (0: bad tree, reported, nothing written), the
// stop node, the number of its children, the residual mass left there.
struct WalkOut { int32_t* path; int32_t* out_tok; int32_t* excl; float* excl_p; };
struct WalkEnd { int na, stop, n_excl; float R; };

__device__ __forceinline__ WalkEnd sampled_walk(const sd_batch& bt, int b, int lane, const int32_t* __restrict__ draft,
                                                const float* p_child, const float* __restrict__ u, const WalkOut& o,
                                                int32_t* status) {
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
        if (lane == 0) set_status(status, SD_ERR_INVALID_TREE);
        return WalkEnd{0, 0, 0, 0.f};
    }
    // parent, token, probability and uniform number of the (up to) two nodes this lane looks after
    const bool has0 = lane < n, has1 = lane + 32 < n;
    const int pa0 = has0 ? par[lane] : -2, pa1 = has1 ? par[lane + 32] : -2;
    const int tk0 = has0 ? dt[lane] : -1, tk1 = has1 ? dt[lane + 32] : -1;
    const float pc0 = has0 ? p_child[(size_t)b * T + lane] : 0.f, pc1 = has1 ? p_child[(size_t)b * T + lane + 32] : 0.f;
    const float u0 = has0 ? u[(size_t)b * T + lane] : 0.f, u1 = has1 ? u[(size_t)b * T + lane + 32] : 0.f;
    int cur = 0, na = 1;
    float R = 1.f;
    if (lane == 0) o.path[0] = 0;
    while (true) {
        // children of cur, as a 64-bit mask in node order
        const uint32_t lo = __ballot_sync(0xffffffffu, pa0 == cur), hi = __ballot_sync(0xffffffffu, pa1 == cur);
        uint64_t kids = ((uint64_t)hi << 32) | lo;
        R = 1.f;
        int nxt = -1, nxt_tok = -1;
        while (kids) {                                       // warp-uniform loop
            const int c = __ffsll((long long)kids) - 1;
            kids &= kids - 1;
            const int tc = __shfl_sync(0xffffffffu, c < 32 ? tk0 : tk1, c & 31);
            const float pc = __shfl_sync(0xffffffffu, c < 32 ? pc0 : pc1, c & 31);
            const float uc = __shfl_sync(0xffffffffu, c < 32 ? u0 : u1, c & 31);
            // siblings must carry distinct tokens (an earlier sibling's rejection already removed the mass)
            if (__any_sync(0xffffffffu, (pa0 == cur && lane < c && tk0 == tc) || (pa1 == cur && lane + 32 < c && tk1 == tc)))
                if (lane == 0) set_status(status, SD_ERR_INVALID_ARG);
            if (uc * R < pc) { nxt = c; nxt_tok = tc; break; }
            R -= pc;
        }
        if (nxt < 0) break;
        if (lane == 0) { o.path[na] = nxt; o.out_tok[na - 1] = nxt_tok; }
        cur = nxt;
        ++na;
    }
    // the stop node's drafted tokens carry no mass in the residual
    const uint32_t lo = __ballot_sync(0xffffffffu, pa0 == cur), hi = __ballot_sync(0xffffffffu, pa1 == cur);
    const int rank0 = __popc(lo & ((1u << lane) - 1u)), rank1 = __popc(lo) + __popc(hi & ((1u << lane) - 1u));
    if (pa0 == cur) { o.excl[rank0] = tk0; o.excl_p[rank0] = pc0; }
    if (pa1 == cur) { o.excl[rank1] = tk1; o.excl_p[rank1] = pc1; }
    for (int k = na - 1 + lane; k < T; k += 32) { if (k >= na) o.path[k] = -1; o.out_tok[k] = -1; }
    return WalkEnd{na, cur, __popc(lo) + __popc(hi), R};
}

// one warp per sequence
__global__ void sampled_walk_kernel(sd_batch bt, const int32_t* __restrict__ draft, const float* __restrict__ p_child,
                                    const float* __restrict__ u, int32_t* n_acc, int32_t* path, int32_t* out_tok,
                                    int32_t* new_len, float* resid, int32_t* stop_row, int32_t* n_excl, int32_t* excl,
                                    float* excl_p, int32_t* status) {
    const int b = blockIdx.x, lane = threadIdx.x;
    const int T = bt.T_max;
    const WalkOut o{path + (size_t)b * T, out_tok + (size_t)b * T, excl + (size_t)b * 64, excl_p + (size_t)b * 64};
    const WalkEnd e = sampled_walk(bt, b, lane, draft, p_child, u, o, status);
    if (lane == 0) {
        n_acc[b] = e.na;
        n_excl[b] = e.n_excl;
        stop_row[b] = b * T + e.stop;
        resid[b] = e.R;
        if (e.na > 0) new_len[b] = bt.len[b] + e.na;
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

// grid (blocks of 256 tokens, sequences): the stop node's row becomes the residual it is drawn from, then
// the block's masses are summed in a fixed order (pairwise tree over the 256 positions).  Point-mass
// drafts (q_rows null): the drafted tokens of the stop node lose their mass.  Drafts sampled from a
// distribution (chains): where a draft was rejected (n_excl[b] != 0) the mass becomes
// max(p - q, 0) with q = the draft's distribution behind the stop node, row stop_row[b] of q_rows.
// With `logits` (the LM-head pass kept its raw logits: chain decoding, few rows) the stop row's
// probabilities are formed here, exp(logit / temperature - lse), instead of by a second pass over W.
__global__ void __launch_bounds__(kResBlock)
residual_blocksum_kernel(int V, const int32_t* __restrict__ n_excl, const int32_t* __restrict__ excl,
                         const float* __restrict__ q_rows, const int32_t* __restrict__ stop_row,
                         const float* __restrict__ logits, const float* __restrict__ lse, float inv_temp,
                         float* __restrict__ mass, float* __restrict__ block_sum, int n_blocks) {
    __shared__ float s_v[kResBlock];
    const int b = blockIdx.y;
    const int t = blockIdx.x * kResBlock + threadIdx.x;
    float m = 0.f;
    if (t < V) {
        if (logits) {
            const int row = stop_row[b];
            m = __expf(__ldg(logits + (size_t)row * V + t) * inv_temp - __ldg(lse + row));
            if (!q_rows || !n_excl[b]) mass[(size_t)b * V + t] = m;
        } else {
            m = mass[(size_t)b * V + t];
        }
        const int ne = n_excl[b];
        if (q_rows) {
            if (ne) {
                m = fmaxf(m - __ldg(q_rows + (size_t)stop_row[b] * V + t), 0.f);
                mass[(size_t)b * V + t] = m;
            }
        } else {
            bool hit = false;
            for (int e = 0; e < ne; ++e) hit |= (__ldg(excl + (size_t)b * 64 + e) == t);
            if (hit) { m = 0.f; mass[(size_t)b * V + t] = 0.f; }
        }
    }
    s_v[threadIdx.x] = m;
    __syncthreads();
    for (int d = kResBlock / 2; d >= 1; d >>= 1) {
        if (threadIdx.x < d) s_v[threadIdx.x] += s_v[threadIdx.x + d];
        __syncthreads();
    }
    if (threadIdx.x == 0) block_sum[(size_t)b * n_blocks + blockIdx.x] = s_v[0];
}

// Where the running sum *acc_io + v[0] + v[1] + ... first reaches `target`, among the elements with
// v > 0 (all v >= 0), found by one warp in a few rounds: the range is cut into 32 consecutive pieces,
// every lane sums one, an inclusive scan over the lanes gives each piece's end value, and the search
// goes on inside the first piece that has mass and whose end value reaches the target, until the
// pieces are single elements.  Every addition happens in a fixed order, so the answer is the same in
// every run.  Returns the index, or -1 when the whole sum stays short; *acc_io then holds the running
// sum in front of the returned element (all of it for -1); *last_pos the last index with v > 0, if any.
// One level down the same elements are added in smaller pieces: where that leaves the refined search
// a rounding short of the target, the piece's last element with mass is the answer.
__device__ __forceinline__ int warp_find_crossing(const float* v, int n, float target, float* acc_io, int* last_pos, int lane) {
    int lo = 0, hi = n;
    float base = *acc_io;
    for (bool top = true;; top = false) {
        const int chunk = (hi - lo + 31) / 32;
        const int i0 = min(hi, lo + lane * chunk), i1 = min(hi, i0 + chunk);
        float sum = 0.f;
        int lastp = -1;
        for (int i = i0; i < i1; ++i) {
            const float x = v[i];
            sum += x;
            if (x > 0.f) lastp = i;
        }
        float incl = sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const float y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        float excl = __shfl_up_sync(0xffffffffu, incl, 1);
        if (lane == 0) excl = 0.f;
        const int lp = __reduce_max_sync(0xffffffffu, lastp);
        if (top && last_pos && lp >= 0) *last_pos = lp;
        const uint32_t cand = __ballot_sync(0xffffffffu, sum > 0.f && base + incl >= target);
        if (!cand) {
            const float all = base + __shfl_sync(0xffffffffu, incl, 31);
            if (top) { *acc_io = all; return -1; }
            *acc_io = all - v[lp];                                   // (lp >= 0: the piece was chosen for having mass)
            return lp;
        }
        const int L0 = __ffs(cand) - 1;
        base += __shfl_sync(0xffffffffu, excl, L0);
        lo = __shfl_sync(0xffffffffu, i0, L0);
        hi = __shfl_sync(0xffffffffu, i1, L0);
        if (chunk == 1) { *acc_io = base; return lo; }
    }
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
        warp_find_crossing(s_bs, n_blocks, INFINITY, &total, nullptr, lane);
        const float target = w[b] * total;
        float acc = 0.f;
        int k = warp_find_crossing(s_bs, n_blocks, target, &acc, nullptr, lane);
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
            const int i = warp_find_crossing(s_m, kResBlock, s_target, &acc, &lastp, lane);
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

// Residual draw from the LM-head pass's own statistics, by one CTA of 256 threads for one sequence.
// The masses of the 32-row vocabulary groups of the stop row follow from (group maximum, group sum)
// and the row's lse; the drafted children's probabilities are taken out of their groups; warp 0 finds
// the group in which the cumulative mass reaches w * (total); that group's 32 logits are recomputed
// (32 dot products) and the token is found among them.  W is not streamed a second time and no
// logits-sized data exist.  row: LM-head row of the stop node; excl / excl_p: its ne drafted children.
constexpr int kPickMaxGroups = 8192;   // vocabularies up to 262144 tokens
// kClusterCtas > 1: the CTAs of the cluster share the reading of the table (each entry sits in a
// sector of its own, so one SM's load path is the limit) and push the masses into the shared memory
// of the cluster's first CTA, which alone goes on; every CTA of the cluster must make the call.
template <int kClusterCtas>
__device__ __forceinline__ void residual_pick_groups(const uint16_t* __restrict__ hidden, const uint16_t* __restrict__ W,
                                                     int Hd, int V, float inv_temp, float row_lse, int M, int row,
                                                     const float2* __restrict__ group_stats, int n_groups, float wb,
                                                     int ne, const int32_t* excl, const float* excl_p,
                                                     int32_t* out_slot, int32_t* status) {
    __shared__ float s_g[kPickMaxGroups];
    __shared__ float s_part[256];                                      // sums of the threads' runs of groups
    __shared__ float s_m[32];
    __shared__ int32_t s_ex[64];                                       // the stop node's drafted tokens ...
    __shared__ float s_exp[64];                                        // ... and their probabilities
    __shared__ float s_acc, s_target;
    __shared__ int s_k, s_pick, s_last;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float c2 = inv_temp * 1.4426950408889634f;
    const float lse2 = row_lse * 1.4426950408889634f;
    {
        // (one 8-byte entry per group, a table row apart: the loads of a batch are issued together)
        const int rank = kClusterCtas > 1 ? (int)sm100::cluster_ctarank() : 0;
        const int per_cta = (n_groups + kClusterCtas - 1) / kClusterCtas;
        const int g_end = min(n_groups, (rank + 1) * per_cta);
        const uint32_t dst = kClusterCtas > 1 ? sm100::map_dsmem(sm100::smem_u32(s_g), 0) : 0;
        constexpr int kAhead = 8;
        for (int g0 = rank * per_cta + threadIdx.x; g0 < g_end; g0 += (int)blockDim.x * kAhead) {
            float2 st[kAhead];
#pragma unroll
            for (int a = 0; a < kAhead; ++a) {
                const int g = g0 + (int)blockDim.x * a;
                if (g < g_end) st[a] = __ldg(group_stats + (size_t)g * M + row);
            }
#pragma unroll
            for (int a = 0; a < kAhead; ++a) {
                const int g = g0 + (int)blockDim.x * a;
                if (g < g_end) {
                    const float m = st[a].y > 0.f ? st[a].y * exp2f(st[a].x * c2 - lse2) : 0.f;
                    if (kClusterCtas > 1) sm100::st_dsmem_f32(dst + g * 4, m);
                    else s_g[g] = m;
                }
            }
        }
        if (kClusterCtas > 1) {
            sm100::cluster_arrive_release();
            sm100::cluster_wait_acquire();
            if (rank != 0) return;
        }
    }
    if (threadIdx.x < ne) { s_ex[threadIdx.x] = excl[threadIdx.x]; s_exp[threadIdx.x] = excl_p[threadIdx.x]; }
    __syncthreads();
    if (threadIdx.x == 0)                                              // drafted children carry no mass (fixed order)
        for (int e = 0; e < ne; ++e) {
            const int g = s_ex[e] >> 5;
            s_g[g] = fmaxf(s_g[g] - s_exp[e], 0.f);
        }
    __syncthreads();
    // every thread sums a run of consecutive groups; the search goes over the 256 sums, then inside one run
    const int run = (n_groups + (int)blockDim.x - 1) / (int)blockDim.x;
    {
        const int g0 = min(n_groups, (int)threadIdx.x * run), g1 = min(n_groups, g0 + run);
        float sum = 0.f;
        for (int g = g0; g < g1; ++g) sum += s_g[g];
        s_part[threadIdx.x] = sum;
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        float total = 0.f;
        warp_find_crossing(s_part, (int)blockDim.x, INFINITY, &total, nullptr, lane);
        const float target = wb * total;
        float acc = 0.f;
        int k = -1;
        const int t = warp_find_crossing(s_part, (int)blockDim.x, target, &acc, nullptr, lane);
        if (t >= 0) {
            const int g0 = t * run, len = min(n_groups, g0 + run) - g0;
            int lastp = -1;
            k = warp_find_crossing(s_g + g0, len, target, &acc, &lastp, lane);
            if (k < 0) { k = max(lastp, 0); acc -= s_g[g0 + k]; }      // a rounding short inside the run: its last group with mass
            k += g0;
        } else {                                                       // no mass anywhere (reported below), or w * total rounded up
            k = n_groups - 1;
            acc -= s_g[k];
        }
        if (lane == 0) { s_acc = acc; s_target = target; s_k = k; s_pick = -1; s_last = -1; }
    }
    __syncthreads();
    const uint4* hrow = reinterpret_cast<const uint4*>(hidden + (size_t)row * Hd);
    // the 32 probabilities of group k, recomputed into s_m: eight warps, four tokens each
    auto recompute_group = [&](int k) {
        const int t0 = k * 32 + warp * 4;
        const uint4* wrow[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) wrow[i] = reinterpret_cast<const uint4*>(W + (size_t)min(t0 + i, V - 1) * Hd);
        float l[4];
        warp_dots_bf16<4>(wrow, hrow, Hd / 8, lane, l);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int t = t0 + i;
            bool hit = false;
            for (int e = lane; e < ne; e += 32) hit |= (s_ex[e] == t);
            const float m = (t >= V || __any_sync(0xffffffffu, hit)) ? 0.f : __expf(l[i] * inv_temp - row_lse);
            if (lane == 0) s_m[warp * 4 + i] = m;
        }
        __syncthreads();
    };
    for (int k = s_k; k < n_groups; ++k) {
        recompute_group(k);
        if (threadIdx.x < 32) {
            float acc = s_acc;
            int lastp = -1;
            const int i = warp_find_crossing(s_m, 32, s_target, &acc, &lastp, lane);
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
        *out_slot = pick;
    }
}

// one CTA per sequence
__global__ void __launch_bounds__(256)
residual_pick_groups_kernel(sd_batch bt, const uint16_t* __restrict__ hidden, const uint16_t* __restrict__ W, int Hd, int V,
                            float inv_temp, const float* __restrict__ lse, const float2* __restrict__ group_stats, int n_groups,
                            const float* __restrict__ w, const int32_t* __restrict__ stop_row, const int32_t* __restrict__ n_excl,
                            const int32_t* __restrict__ excl, const float* __restrict__ excl_p, const int32_t* __restrict__ n_acc,
                            int32_t* out_tok, int32_t* status) {
    const int b = blockIdx.x;
    const int na = n_acc[b];
    if (na < 1 || na > bt.T_max) return;                               // bad tree: already reported
    const int row = stop_row[b];
    residual_pick_groups<1>(hidden, W, Hd, V, inv_temp, lse[row], bt.B * bt.T_max, row, group_stats, n_groups, w[b], n_excl[b],
                            excl + (size_t)b * 64, excl_p + (size_t)b * 64, out_tok + (size_t)b * bt.T_max + na - 1, status);
}

// Chains drafted by SAMPLING from a draft distribution (one warp per sequence): node j's token is kept
// iff u * q(token) < p(token), q and p the draft's and the target's probability of that token behind
// node j - 1; the walk stops at the first rejection.  Leaves the accepted prefix, the stop node's
// LM-head row and whether a draft was rejected there (the residual then is max(p - q, 0), else p).
__global__ void chain_walk_q_kernel(sd_batch bt, const int32_t* __restrict__ draft, const float* __restrict__ p_child,
                                    const float* __restrict__ q_tok, const float* __restrict__ u, int32_t* n_acc,
                                    int32_t* path, int32_t* out_tok, int32_t* new_len, int32_t* stop_row, int32_t* rejected,
                                    int32_t* status) {
    const int b = blockIdx.x, lane = threadIdx.x;
    const int T = bt.T_max;
    const int n = bt.n_nodes[b];
    const int32_t* par = bt.parents + (size_t)b * T;
    const int32_t* dt = draft + (size_t)b * T;
    bool bad = (n < 1 || n > T), branching = false;
    if (!bad)
        for (int i = lane; i < n; i += 32) {
            const int p = par[i];
            if (i == 0 ? (p != -1) : (p < 0 || p >= i)) bad = true;
            else if (i > 0 && p != i - 1) branching = true;
        }
    bad = __any_sync(0xffffffffu, bad);
    branching = __any_sync(0xffffffffu, branching);
    if (bad || branching) {
        if (lane == 0) {
            set_status(status, bad ? SD_ERR_INVALID_TREE : SD_ERR_UNSUPPORTED);
            n_acc[b] = 0; stop_row[b] = b * T; rejected[b] = 0;
        }
        return;
    }
    bool keep[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int j = lane + 32 * h;
        keep[h] = true;
        if (j >= 1 && j < n) {
            const size_t at = (size_t)b * T + j;
            keep[h] = u[at] * q_tok[at] < p_child[at];
        }
    }
    const uint32_t lo = __ballot_sync(0xffffffffu, !keep[0]), hi = __ballot_sync(0xffffffffu, !keep[1]);
    const int na = lo ? __ffs(lo) - 1 : (hi ? 32 + __ffs(hi) - 1 : n);      // the first rejected node, or all
    for (int k = lane; k < T; k += 32) {
        path[(size_t)b * T + k] = k < na ? k : -1;
        out_tok[(size_t)b * T + k] = k + 1 < na ? dt[k + 1] : -1;            // slot na - 1: the token still to be drawn
    }
    if (lane == 0) {
        n_acc[b] = na;
        new_len[b] = bt.len[b] + na;
        stop_row[b] = b * T + na - 1;
        rejected[b] = na < n ? 1 : 0;
    }
}

sd_status launch_accept_chain_sampled(const sd_batch& bt, const void* hidden, const void* W, int Hd, int V, float inv_temp,
                                      const float* lse, const float* logits, const int32_t* draft, const float* q_tok,
                                      const float* q_rows, const float* u, const float* w, int32_t* n_acc, int32_t* path,
                                      int32_t* out_tok, int32_t* new_len, void* ws, size_t ws_bytes, int32_t* dev_status,
                                      cudaStream_t st) {
    const int B = bt.B, T = bt.T_max;
    if (Hd > 16384 || (V + kResBlock - 1) / kResBlock > kPickMaxBlocks) return SD_ERR_UNSUPPORTED;
    if (ws_bytes < sampled_workspace_bytes(B, T, V, 16384)) return SD_ERR_WORKSPACE;
    const SampledWs s = carve(ws, B, T, V, 16384);
    const uint16_t* h = static_cast<const uint16_t*>(hidden);
    const uint16_t* Wp = static_cast<const uint16_t*>(W);
    const int n_blocks = (V + kResBlock - 1) / kResBlock;
    child_prob_kernel<<<(B * T * 32 + 127) / 128, 128, 0, st>>>(bt, h, Wp, Hd, V, inv_temp, lse, draft, s.p_child, dev_status);
    chain_walk_q_kernel<<<B, 32, 0, st>>>(bt, draft, s.p_child, q_tok, u, n_acc, path, out_tok, new_len, s.stop_row, s.n_excl,
                                         dev_status);
    if (!logits) {
        // the stop rows' probabilities over the vocabulary: the LM-head kernel once more, in its store mode
        gather_stop_rows_kernel<<<B, 128, 0, st>>>(h, Hd, lse, s.stop_row, s.stop_hidden, s.stop_lse);
        const sd_status ls = launch_lmhead_mass(s.stop_hidden, W, B, Hd, V, inv_temp, s.stop_lse, s.mass, s.lm_ws,
                                                stats_workspace_bytes(B, V), dev_status, st);
        if (ls != SD_OK) return ls;
    }
    // ... turned into the residual max(p - q, 0) where a draft was rejected (with the kept logits of the
    // LM-head pass the probabilities themselves are formed here as well)
    residual_blocksum_kernel<<<dim3(n_blocks, B), kResBlock, 0, st>>>(V, s.n_excl, s.excl, q_rows, s.stop_row, logits, lse,
                                                                      inv_temp, s.mass, s.block_sum, n_blocks);
    residual_pick_kernel<<<B, kResBlock, 0, st>>>(bt, V, w, s.mass, s.block_sum, n_blocks, n_acc, out_tok, dev_status);
    return cuda_ok(cudaGetLastError());
}

// ---------------------------------------------------------------------------
// Trees whose children were SAMPLED, every child of node i independently from the draft's distribution
// q_i: the rule is applied child after child, and every rejection replaces the target distribution r
// by the normalised positive part of r - q_i.  Every r met this way is max(p_i - a q_i, 0) / b with two
// scalars (a = 0, b = 1 at a node's start; a rejection makes a <- a + b, b <- sum_v max(p_i - a q_i, 0)),
// so a rejection costs one reduction over the vocabulary.  One cluster of eight CTAs per sequence:
// every CTA keeps its eighth of p_i (from the logits the LM-head pass kept) and of q_i in shared
// memory while the walk is at node i, sums its part in a fixed order, and the eight partial sums
// are exchanged through remote stores and added in rank order, so that all eight CTAs take the same
// decisions.  The last token is drawn from max(p - a q, 0) by inverse CDF in vocabulary order: the
// CTA whose slice holds the crossing finds it.
// ---------------------------------------------------------------------------
constexpr int kTreeQCluster = 8;
constexpr int kTreeQThreads = 256;
constexpr int kTreeQMaxSlice = 20480;          // vocabulary entries per CTA: V <= 163840

__global__ void __launch_bounds__(kTreeQThreads)
tree_walk_q_kernel(sd_batch bt, int V, float inv_temp, const float* __restrict__ lse, const float* __restrict__ logits,
                   const int32_t* __restrict__ draft, const float* __restrict__ q_rows, const float* __restrict__ u,
                   const float* __restrict__ w, int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                   int32_t* status) {
    extern __shared__ float s_pq[];                 // p slice, then q slice
    __shared__ float s_part[kTreeQThreads];         // sums of the threads' runs
    __shared__ float s_run[128];                    // one run, element by element (the last draw)
    __shared__ float s_cta2[2][kTreeQCluster];      // the eight CTAs' sums, written by their owners; two sets in
                                                    // turn: a CTA may start the next exchange while another still
                                                    // reads this one (it cannot get two ahead: the barrier)
    __shared__ int32_t s_path[kMaxT];
    __shared__ float s_px, s_qx;
    __shared__ int s_bad;
    const int b = blockIdx.x / kTreeQCluster;
    const int rank = (int)sm100::cluster_ctarank();
    const int T = bt.T_max, tid = threadIdx.x, lane = tid & 31;
    const int slice = (V + kTreeQCluster - 1) / kTreeQCluster;
    const int v0 = min(V, rank * slice), v1 = min(V, v0 + slice), len = v1 - v0;
    const int run = (slice + kTreeQThreads - 1) / kTreeQThreads;     // <= 80 entries per thread
    float* s_p = s_pq;
    float* s_q = s_pq + slice;
    const int n = bt.n_nodes[b];
    const int32_t* par = bt.parents + (size_t)b * T;
    const int32_t* dt = draft + (size_t)b * T;
    // the tree, checked by every CTA in the same way
    if (tid == 0) s_bad = 0;
    __syncthreads();
    if (n < 1 || n > T) { if (tid == 0) s_bad = SD_ERR_INVALID_TREE; }
    else
        for (int i = tid; i < n; i += kTreeQThreads) {
            const int p = par[i];
            if (i == 0 ? (p != -1) : (p < 0 || p >= i)) s_bad = SD_ERR_INVALID_TREE;
            else if (i > 0 && (dt[i] < 0 || dt[i] >= V)) atomicCAS(&s_bad, 0, (int)SD_ERR_BOUNDS);
        }
    __syncthreads();
    if (s_bad != 0) {                               // (the same in every CTA: nobody reaches a cluster barrier)
        if (rank == 0 && tid == 0) { set_status(status, s_bad); n_acc[b] = 0; }
        return;
    }
    // sum over this CTA's slice of max(p - a q, 0), every thread a run of consecutive entries; the eight
    // sums are exchanged; returns their total (rank order), the same bits in every CTA
    int n_red = 0;
    const float* s_cta = s_cta2[0];                 // the set of the latest exchange
    auto reduce = [&](float a) -> float {
        float* mine = s_cta2[n_red & 1];
        ++n_red;
        s_cta = mine;
        const int i0 = min(len, tid * run), i1 = min(len, i0 + run);
        float sum = 0.f;
        for (int i = i0; i < i1; ++i) sum += fmaxf(s_p[i] - a * s_q[i], 0.f);
        s_part[tid] = sum;
        __syncthreads();
        if (tid < 32) {
            float total = 0.f;
            warp_find_crossing(s_part, kTreeQThreads, INFINITY, &total, nullptr, lane);
            if (lane < kTreeQCluster)
                sm100::st_dsmem_f32(sm100::map_dsmem(sm100::smem_u32(&mine[rank]), (uint32_t)lane), total);
        }
        sm100::cluster_arrive_release();
        sm100::cluster_wait_acquire();
        float all = 0.f;
#pragma unroll
        for (int r = 0; r < kTreeQCluster; ++r) all += s_cta[r];
        return all;
    };
    int cur = 0, na = 1;
    float a = 0.f, bsum = 1.f;
    if (tid == 0) s_path[0] = 0;
    while (true) {
        // this CTA's slice of p and q behind node cur
        const int row = b * T + cur;
        const float row_lse = lse[row];
        const float* lrow = logits + (size_t)row * V + v0;
        const float* qrow = q_rows + (size_t)row * V + v0;
        for (int i = tid; i < len; i += kTreeQThreads) {
            s_p[i] = __expf(__ldg(lrow + i) * inv_temp - row_lse);
            s_q[i] = __ldg(qrow + i);
        }
        __syncthreads();
        a = 0.f; bsum = 1.f;
        int nxt = -1;
        bool summed = false;                         // the partial sums on hand belong to this node and this a
        for (int c = cur + 1; c < n; ++c) {          // children of cur in node order (the same walk in every CTA)
            if (par[c] != cur) continue;
            const int x = dt[c];
            if (tid == 0) {
                s_px = __expf(__ldg(logits + (size_t)row * V + x) * inv_temp - row_lse);
                s_qx = __ldg(q_rows + (size_t)row * V + x);
            }
            __syncthreads();
            const float num = fmaxf(s_px - a * s_qx, 0.f);
            const bool keep = u[(size_t)b * T + c] * bsum * s_qx < num;
            __syncthreads();                        // (s_px, s_qx are rewritten for the next child)
            if (keep) { nxt = c; break; }
            a += bsum;
            bsum = reduce(a);
            summed = true;
        }
        if (nxt < 0) {
            if (!summed) bsum = reduce(a);           // the sums the draw walks over (nothing rejected here: all of p)
            break;
        }
        if (tid == 0) s_path[na] = nxt;
        cur = nxt;
        ++na;
        __syncthreads();
    }
    // outputs of the walk
    if (rank == 0) {
        for (int k = tid; k < T; k += kTreeQThreads) {
            path[(size_t)b * T + k] = k < na ? s_path[k] : -1;
            if (k != na - 1) out_tok[(size_t)b * T + k] = k + 1 < na ? dt[s_path[k + 1]] : -1;
        }
        if (tid == 0) { n_acc[b] = na; new_len[b] = bt.len[b] + na; }
    }
    // the last token: which CTA's slice holds the crossing of w * (total mass), then which run, then which entry
    const float target = w[b] * bsum;
    float before = 0.f;
    int owner = -1, last_with_mass = -1;
    for (int r = 0; r < kTreeQCluster; ++r) {
        if (s_cta[r] > 0.f) last_with_mass = r;
        if (owner < 0 && s_cta[r] > 0.f && before + s_cta[r] >= target) owner = r;
        if (owner < 0) before += s_cta[r];
    }
    if (owner < 0) {                                 // rounding left the sum short: the last slice with mass
        owner = last_with_mass;
        if (owner >= 0) before -= s_cta[owner];
    }
    if (owner < 0) {                                 // no mass at all (inputs not finite, or r vanished by rounding)
        if (rank == 0 && tid == 0) { set_status(status, SD_ERR_BOUNDS); out_tok[(size_t)b * T + na - 1] = 0; }
        return;
    }
    if (rank != owner) return;
    __shared__ float s_acc;
    __shared__ int s_t, s_pick;
    if (tid < 32) {
        float acc = before;
        int lastp = -1;
        int t = warp_find_crossing(s_part, kTreeQThreads, target, &acc, &lastp, lane);
        if (t < 0) { t = max(lastp, 0); acc -= s_part[t]; }
        if (lane == 0) { s_acc = acc; s_t = t; }
    }
    __syncthreads();
    const int i0 = min(len, s_t * run), i1 = min(len, i0 + run);
    if (tid < i1 - i0) s_run[tid] = fmaxf(s_p[i0 + tid] - a * s_q[i0 + tid], 0.f);
    __syncthreads();
    if (tid < 32) {
        float acc = s_acc;
        int lastp = -1;
        int k = warp_find_crossing(s_run, i1 - i0, target, &acc, &lastp, lane);
        if (k < 0) k = max(lastp, 0);
        if (lane == 0) out_tok[(size_t)b * T + na - 1] = v0 + i0 + k;
    }
}

sd_status launch_accept_tree_sampled_q(const sd_batch& bt, int V, float inv_temp, const float* lse, const float* logits,
                                       const int32_t* draft, const float* q_rows, const float* u, const float* w,
                                       int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                                       int32_t* dev_status, cudaStream_t st) {
    const int slice = (V + kTreeQCluster - 1) / kTreeQCluster;
    if (slice > kTreeQMaxSlice) return SD_ERR_UNSUPPORTED;
    const size_t dyn = (size_t)slice * 2 * sizeof(float);
    if (cudaFuncSetAttribute(tree_walk_q_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return SD_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(bt.B * kTreeQCluster);
    cfg.blockDim = dim3(kTreeQThreads);
    cfg.dynamicSmemBytes = dyn;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kTreeQCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, tree_walk_q_kernel, bt, V, inv_temp, lse, logits, draft, q_rows, u, w, n_acc, path, out_tok,
                           new_len, dev_status) != cudaSuccess)
        return SD_ERR_CUDA;
    return SD_OK;
}

// ---------------------------------------------------------------------------
// Tail of a verify step at a sampling temperature, behind the LM-head tiles of a statistics pass: one
// cluster of eight CTAs per sequence.
//   1. every CTA merges the per-CTA soft-max partials of eight of the sequence's LM-head rows -> lse
//   2. every warp of the cluster computes one node's probability under its parent's distribution
//   3. every CTA repeats the (cheap) rejection walk into its own shared memory
//   4. the cluster's first CTA writes the outputs and draws the last token from the group table
//   5. every CTA copies the accepted nodes' K/V into the caches of its share of the layers
// Steps 1 and 2 hand their results on through global memory across a cluster barrier.  The arithmetic
// is that of the stand-alone kernels (the same device functions), so the results are the same bits.
// ---------------------------------------------------------------------------
constexpr int kTailCluster = 8;
__global__ void __launch_bounds__(256)
sampled_tail_kernel(sd_batch bt, const __grid_constant__ CompactLayers ly, int L, LmTables tb, float c2,
                    const uint16_t* __restrict__ hidden, const uint16_t* __restrict__ W, int Hd, int V, float inv_temp,
                    const float2* __restrict__ group_stats, int n_groups, const int32_t* __restrict__ draft,
                    const float* __restrict__ u, const float* __restrict__ w, float* lse, float* p_child,
                    int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len, int32_t* status) {
    __shared__ int32_t s_path[kMaxT], s_tok[kMaxT], s_excl[64];
    __shared__ float s_excl_p[64];
    __shared__ WalkEnd s_end;
    const int b = blockIdx.x / kTailCluster;
    const int rank = (int)sm100::cluster_ctarank();
    const int T = bt.T_max, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // 1. lse of rows rank * 8 .. + 7 (of every 64): eight lanes per row, the first two warps
    if (warp < 2)
        for (int r0 = 0; r0 < T; r0 += 8 * kTailCluster) {
            const int node = r0 + rank * 8 + (threadIdx.x >> 3), sub = threadIdx.x & 7;
            int32_t k, i;
            const float row_lse = merge_row_stats(tb.part_key, tb.part_idx, tb.part_ref, tb.part_sum, tb.n_ctas, kLmMaxCols,
                                                  b * T + node, node < T, sub, c2, k, i);
            if (node < T && sub == 0) lse[b * T + node] = row_lse;
        }
    sm100::cluster_arrive_release();
    sm100::cluster_wait_acquire();
    // 2. probabilities of the drafted tokens: node rank * 8 + warp (of every 64)
    for (int j0 = 0; j0 < T; j0 += 8 * kTailCluster) {
        const int j = j0 + rank * 8 + warp;
        if (j < T) {
            const float p = child_prob(bt, b, j, lane, hidden, W, Hd, V, inv_temp, lse, draft, status);
            if (lane == 0) p_child[(size_t)b * T + j] = p;
        }
    }
    sm100::cluster_arrive_release();
    sm100::cluster_wait_acquire();
    // 3. the walk
    if (warp == 0) {
        const WalkOut o{s_path, s_tok, s_excl, s_excl_p};
        const WalkEnd e = sampled_walk(bt, b, lane, draft, p_child, u, o, status);
        if (lane == 0) s_end = e;
    }
    __syncthreads();
    const WalkEnd e = s_end;
    // 4. outputs and the last token (the whole cluster reads the group table, the first CTA draws)
    if (rank == 0 && threadIdx.x == 0) {
        n_acc[b] = e.na;
        if (e.na > 0) new_len[b] = bt.len[b] + e.na;
    }
    if (e.na > 0) {                                                    // (the same in every CTA of the cluster)
        if (rank == 0)
            for (int k = threadIdx.x; k < T; k += blockDim.x) {
                path[(size_t)b * T + k] = s_path[k];
                if (k != e.na - 1) out_tok[(size_t)b * T + k] = s_tok[k];
            }
        const int row = b * T + e.stop;
        residual_pick_groups<kTailCluster>(hidden, W, Hd, V, inv_temp, lse[row], bt.B * T, row, group_stats, n_groups, w[b],
                                           e.n_excl, s_excl, s_excl_p, out_tok + (size_t)b * T + e.na - 1, status);
    }
    // 5. accepted rows into the caches; the first CTA, busy with the draw, takes the smallest share
    for (int l = kTailCluster - 1 - rank; l < L; l += kTailCluster)
        compact_sequence(bt, ly, l, 1, b, e.na, s_path, threadIdx.x, blockDim.x, status);
}

sd_status launch_lmhead_accept_sampled_compact(const sd_batch& bt, const void* hidden, const void* W, int Hd, int V,
                                               float inv_temp, const int32_t* draft, const float* u, const float* w,
                                               const sd_kv_layer* layers, int L, const void* const* kt, const void* const* vt,
                                               float* lse, float* group_stats, int32_t* n_acc, int32_t* path,
                                               int32_t* out_tok, int32_t* new_len, void* ws, size_t ws_bytes,
                                               int32_t* dev_status, cudaStream_t st) {
    const int B = bt.B, T = bt.T_max, M = B * T;
    if (Hd > 16384 || (V + 31) / 32 > kPickMaxGroups) return SD_ERR_UNSUPPORTED;
    if (ws_bytes < sampled_workspace_bytes(B, T, V, 16384)) return SD_ERR_WORKSPACE;
    const SampledWs s = carve(ws, B, T, V, 16384);
    const size_t lm_bytes = stats_workspace_bytes(M, V);
    if (M > kLmMaxCols || L > kLayersPerLaunch) {
        // shapes beyond one pass of the candidate tables or one set of layer descriptors: the same steps
        // as separate launches
        sd_status r = launch_lmhead_stats(hidden, W, M, Hd, V, inv_temp, nullptr, nullptr, lse, group_stats, s.lm_ws, lm_bytes,
                                          dev_status, st);
        if (r != SD_OK) return r;
        r = launch_accept_sampled(bt, hidden, W, Hd, V, inv_temp, lse, group_stats, draft, u, w, n_acc, path, out_tok, new_len,
                                  ws, ws_bytes, dev_status, st);
        if (r != SD_OK) return r;
        return launch_compact(bt, layers, L, kt, vt, n_acc, path, dev_status, st);
    }
    LmTables tb;
    const sd_status r = launch_lmhead_stats_tiles(hidden, W, M, Hd, V, inv_temp, lse, group_stats, s.lm_ws, lm_bytes,
                                                  dev_status, st, &tb);
    if (r != SD_OK) return r;
    CompactLayers ly;
    fill_compact_layers(&ly, layers, kt, vt, 0, L);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(B * kTailCluster);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kTailCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float c2 = inv_temp * 1.4426950408889634f;
    const int n_groups = (V + 31) / 32;
    if (cudaLaunchKernelEx(&cfg, sampled_tail_kernel, bt, ly, L, tb, c2, static_cast<const uint16_t*>(hidden),
                           static_cast<const uint16_t*>(W), Hd, V, inv_temp, reinterpret_cast<const float2*>(group_stats),
                           n_groups, draft, u, w, lse, s.p_child, n_acc, path, out_tok, new_len, dev_status) != cudaSuccess)
        return SD_ERR_CUDA;
    return SD_OK;
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
    residual_blocksum_kernel<<<dim3(n_blocks, B), kResBlock, 0, st>>>(V, s.n_excl, s.excl, nullptr, nullptr, nullptr, nullptr, 0.f,
                                                                      s.mass, s.block_sum, n_blocks);
    residual_pick_kernel<<<B, kResBlock, 0, st>>>(bt, V, w, s.mass, s.block_sum, n_blocks, n_acc, out_tok, dev_status);
    return cuda_ok(cudaGetLastError());
}

}  // namespace sdv
