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

// Final step of a clustered launch.  Each CTA of the cluster finishes 128 / NCH rows of the tile: a
// warp takes a few rows at a time, every lane four output columns, and adds up the chunks in chunk
// order (so the result does not depend on timing).  A row of a parked tile is one contiguous
// 512-byte line of the owning CTA's shared memory; all loads of a batch of rows are issued before
// any of them is used, so that their latencies overlap.
struct MergeCtx {
    const sd_batch& bt; const AttnPlan& plan; __nv_bfloat16* out; float* lse;
    uint32_t xo_addr, xs_addr;
    int chunk, rt, b, kvh, n, tpc, tiles_total, warp, lane;
};

template <int NCH>
__device__ __forceinline__ void merge_rows(const MergeCtx& x) {
    constexpr int kRowsPer = kRowTile / NCH;
    constexpr int kBatch = 16 / NCH;                // rows in flight per warp
    const int G = x.bt.Hq / x.bt.Hkv;
    for (int i0 = x.warp * kBatch; i0 < kRowsPer; i0 += 4 * kBatch) {
        float mc[kBatch][NCH], lc[kBatch][NCH];
        float4 v[kBatch][NCH];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int r = x.chunk * kRowsPer + i0 + u;
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                const bool live = (c == NCH - 1) || (c * x.tpc < x.tiles_total);   // that chunk had key tiles
                mc[u][c] = -INFINITY; lc[u][c] = 0.f; v[u][c] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (live && c == x.chunk) {                  // this CTA's own chunk: plain shared-memory reads
                    mc[u][c] = ld_smem_f32(x.xs_addr + r * 4);
                    lc[u][c] = ld_smem_f32(x.xs_addr + (kRowTile + r) * 4);
                    v[u][c] = ld_smem_v4(x.xo_addr + (uint32_t)(r * kD + ((x.lane ^ (r & 31)) << 2)) * 4);
                } else if (live) {
                    mc[u][c] = ld_dsmem_f32(map_dsmem(x.xs_addr + r * 4, c));
                    lc[u][c] = ld_dsmem_f32(map_dsmem(x.xs_addr + (kRowTile + r) * 4, c));
                    v[u][c] = ld_dsmem_v4(map_dsmem(x.xo_addr + (uint32_t)(r * kD + ((x.lane ^ (r & 31)) << 2)) * 4, c));
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int r = x.chunk * kRowsPer + i0 + u;
            const int row = x.rt * kRowTile + r;
            if (row >= x.plan.rows) continue;
            const int node = row / G;
            const int g = row - node * G;
            const size_t orow = ((size_t)x.b * x.bt.T_max + node) * x.bt.Hq + x.kvh * G + g;
            uint2* dst = reinterpret_cast<uint2*>(x.out + orow * kD + x.lane * 4);
            if (node >= x.n) {                               // unused node: zero row
                *dst = make_uint2(0, 0);
                if (x.lse && x.lane == 0) x.lse[orow] = 0.f;
                continue;
            }
            float M = mc[u][0];
#pragma unroll
            for (int c = 1; c < NCH; ++c) M = fmaxf(M, mc[u][c]);
            float den = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                const float w = exp2f(mc[u][c] - M);         // 0 for a chunk without tiles (m = -inf)
                den = fmaf(w, lc[u][c], den);
                acc.x = fmaf(w, v[u][c].x, acc.x); acc.y = fmaf(w, v[u][c].y, acc.y);
                acc.z = fmaf(w, v[u][c].z, acc.z); acc.w = fmaf(w, v[u][c].w, acc.w);
            }
            const float inv = 1.f / den;
            __nv_bfloat162 h0 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
            __nv_bfloat162 h1 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
            *dst = make_uint2(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1));
            if (x.lse && x.lane == 0) x.lse[orow] = (M + log2f(den)) * 0.6931471805599453f;
        }
    }
}


// one launch of `z_count` (sequence rank, layer, KV head) groups starting at plan.z0
template <int NL>
sd_status launch_rows1(const AttnLayers<NL>& layers, const sd_batch& bt, float scale, const AttnPlan& plan,
                       int z_count, int32_t* dev_status, cudaStream_t st);     // one row tile per CTA, 64-key tiles

}  // namespace sdv
