// Pieces of the tree-attention kernel that its launcher shares with it: launch plan, per-layer
// descriptors, and the in-cluster merge of key chunks through distributed shared memory.
#pragma once
#include <stdlib.h>
#include "common.cuh"
#include "sm100.cuh"

namespace sdv {
using namespace sm100;

constexpr int kRowTile = 128;                  // query rows per row tile (MMA M)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;      // log2 units
constexpr int kMaxChunks = 8;                  // = portable cluster size
constexpr int kSplitRounds = 8;                // launches of fewer whole rounds get their remainder as a chunked launch

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct AttnPlan {
    int n_chunks;      // key chunks per sequence (the last one also takes the tree tile)
    int rows;          // T_max * G
    int row_tiles;
    int ctas_per_group;// CTAs along blockIdx.y per (layer, sequence, KV head): row tiles, or pairs of row tiles
    int n_layers;      // layers of this launch
    int ranked;        // dispatch the sequences longest first (only matters when the grid runs in several waves)
    int z0;            // first (sequence rank, layer, KV head) index of this launch: blockIdx.z counts from here
    long long wait_cycles;   // bound of every barrier wait, in SM cycles
    int withhold;      // test hook: the softmax warps never report their first tile, so that a wait runs out
};

// Everything the CTAs of one layer need.  A launch covers up to kMaxLayersPerLaunch layers (the
// descriptors travel as kernel parameters); blockIdx.z enumerates (sequence, layer, KV head).
struct AttnLayer {
    CUtensorMap k_cache, v_cache;   // 2-D [num_blocks*Hkv*64][128], box 64 x 64
    CUtensorMap k_tree, v_tree;     // 3-D (128, Hkv, B*T_max), box 64 x 1 x 64
    const uint16_t* q;              // bf16 [B][T_max][Hq][D]
    __nv_bfloat16* out;             // bf16 [B][T_max][Hq][D]
    float* lse;                     // f32  [B][T_max][Hq] or null
    int32_t num_blocks;
};
constexpr int kMaxLayersPerLaunch = 32;
template <int NL>
struct AttnLayers { AttnLayer l[NL]; };

// Final step of a clustered launch.  Chunk c's CTA has PUSHED its unnormalised rows (and their
// maximum and sum) into the shared memory of the CTA that finishes them: the CTA of chunk o owns rows
// o * 128 / NCH .. of the tile and holds, for each of its rows, one slot per chunk (slot = c * rows
// per CTA + local row).  Every read here is local.  A warp takes a few rows at a time, every lane
// four output columns, and adds up the chunks in chunk order (so the result does not depend on
// timing).  A slot is one contiguous 512-byte line whose 16-byte pieces are XOR-swizzled by the slot
// index (the pushing threads write one row each: without the swizzle a warp's stores would meet in
// one bank group).
struct MergeCtx {
    const sd_batch& bt; const AttnPlan& plan; __nv_bfloat16* out; float* lse;
    uint32_t xo_addr, xs_addr;          // this CTA's exchange area: rows, then maxima [128] and sums [128]
    int chunk, rt, b, kvh, n, tpc, tiles_total, warp, lane;
};

template <int NCH>
__device__ __forceinline__ void merge_rows(const MergeCtx& x) {
    // Eight lanes per row (16 output columns each), four rows per warp at a time; the warp's rows are
    // consecutive, so node and head within the group are counted up instead of divided out.
    constexpr int kRowsPer = kRowTile / NCH;        // rows this CTA finishes
    constexpr int kPerWarp = kRowsPer / 4;          // ... and each of its four warps (a multiple of 4)
    const int G = x.bt.Hq / x.bt.Hkv;
    const int sub = x.lane >> 3, ql = x.lane & 7;
    const int first = x.rt * kRowTile + x.chunk * kRowsPer + x.warp * kPerWarp + sub;   // this lane's first row
    int node = first / G;
    int g = first - node * G;
    // (unrolled: the groups are independent, and one warp per scheduler partition has nothing else to
    //  hide the latency of a group's dependent loads, exponentials and stores behind)
#pragma unroll
    for (int i = 0; i < kPerWarp; i += 4) {
        const int rl = x.warp * kPerWarp + i + sub;             // row among this CTA's rows
        const int row = first + i;
        const bool has_data = row < x.plan.rows && node < x.n;  // only such rows were pushed
        float mc[NCH];
        float M = -INFINITY;
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            const bool live = has_data && ((c == NCH - 1) || (c * x.tpc < x.tiles_total));   // that chunk had key tiles
            mc[c] = live ? ld_smem_f32(x.xs_addr + (c * kRowsPer + rl) * 4) : -INFINITY;
            M = fmaxf(M, mc[c]);
        }
        float den = 0.f;
        float4 acc[4];
#pragma unroll
        for (int p = 0; p < 4; ++p) acc[p] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            if (mc[c] == -INFINITY) continue;                    // a chunk without tiles
            const int slot = c * kRowsPer + rl;
            const float w = ex2_approx(mc[c] - M);
            den = fmaf(w, ld_smem_f32(x.xs_addr + (kRowTile + slot) * 4), den);
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                const float4 v = ld_smem_v4(x.xo_addr + (uint32_t)(slot * kD + (((ql * 4 + p) ^ (slot & 31)) << 2)) * 4);
                acc[p].x = fmaf(w, v.x, acc[p].x); acc[p].y = fmaf(w, v.y, acc[p].y);
                acc[p].z = fmaf(w, v.z, acc[p].z); acc[p].w = fmaf(w, v.w, acc[p].w);
            }
        }
        if (row < x.plan.rows) {
            const size_t orow = ((size_t)x.b * x.bt.T_max + node) * x.bt.Hq + x.kvh * G + g;
            uint4* dst = reinterpret_cast<uint4*>(x.out + orow * kD + ql * 16);
            if (node >= x.n) {                                   // unused node: zero row
                dst[0] = make_uint4(0, 0, 0, 0);
                dst[1] = make_uint4(0, 0, 0, 0);
                if (x.lse && ql == 0) x.lse[orow] = 0.f;
            } else {
                const float inv = __frcp_rn(den);
                uint32_t w[8];
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    __nv_bfloat162 h0 = __floats2bfloat162_rn(acc[p].x * inv, acc[p].y * inv);
                    __nv_bfloat162 h1 = __floats2bfloat162_rn(acc[p].z * inv, acc[p].w * inv);
                    w[2 * p] = *reinterpret_cast<uint32_t*>(&h0);
                    w[2 * p + 1] = *reinterpret_cast<uint32_t*>(&h1);
                }
                dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
                if (x.lse && ql == 0) x.lse[orow] = (M + __log2f(den)) * 0.6931471805599453f;
            }
        }
        g += 4;                                                  // the next group's row: four further on
        while (g >= G) { g -= G; ++node; }
    }
}

// one launch of `z_count` (sequence rank, layer, KV head) groups starting at plan.z0
template <int NL>
sd_status launch_rows1(const AttnLayers<NL>& layers, const sd_batch& bt, float scale, const AttnPlan& plan,
                       int z_count, int32_t* dev_status, cudaStream_t st);     // one row tile per CTA, 64-key tiles

}  // namespace sdv
