// Tree-masked GQA attention for more than 128 query rows per KV head (e.g. 60 nodes x 7 grouped
// heads = 420 rows): two 128-row tiles per CTA, one CTA per SM, 128-key tiles.
//
// The tensor cores of an SM are kept busy by alternating between the two row tiles: while the
// softmax warps of tile A turn their scores into probabilities, the tensor cores run P.V and the
// next score tile of tile B, and the other way round.  Every K/V tile is fetched into shared memory
// once for both row tiles, and a score tile spans 128 keys (two 64-token cache blocks), because a
// tcgen05.mma with both operands in shared memory only runs at the full rate from N = 128 on: at
// N = 64 re-reading the 128 x 16 slice of Q for every instruction takes longer than the arithmetic.
//
// Tensor memory (512 columns): O_A 0..127 | O_B 128..255 | S_A 256..383 | S_B 384..511; the bf16
// probabilities overwrite the first 64 columns of the score tile they were computed from, and feed
// the second MMA from there.  Warps 0-3: softmax of row tile A (one thread per row = one TMEM lane),
// warps 4-7: row tile B, warp 8: TMA producer (one thread; the warp also allocates tensor memory),
// warp 9: ONE thread, the MMA issuer.
//
// The key tiles of a CTA are the 64-token cache blocks of its key chunk, taken two at a time, with
// the tree's own keys as one more block behind the last chunk's prefix blocks (masked per row by the
// node's ancestor bitmask).  A last tile of a single block runs N = 64 score MMAs and half the P.V
// steps.  With several key chunks the chunks of a CTA's row tiles form a thread-block cluster and
// merge their (max, sum, unnormalised O) through distributed shared memory in a fixed order.
#include "attention_shared.cuh"

namespace sdv {

constexpr int kPpThreads = 8 * 32 + 32 + 1;    // 8 softmax warps, TMA warp, one-thread MMA warp
constexpr int kPpTmaWarp = 8, kPpMmaWarp = 9;
constexpr int kPpHalf = 128 * 128;             // bytes of one D-half of a 128-key K/V tile or a 128-row Q tile (16 KiB)
constexpr int kPpBlockHalf = 64 * 128;         // one cache block's share of it (8 KiB)
constexpr int kPpStage = 2 * kPpHalf;          // a K (or V) tile of 128 keys, or the Q of one row tile (32 KiB)
constexpr int kPpKStages = 2, kPpVStages = 2;
constexpr int kPpQBytes = 2 * kPpStage;        // Q of row tiles A and B
constexpr int kPpSmem = kPpQBytes + (kPpKStages + kPpVStages) * kPpStage + 512;
constexpr int kPpTmemCols = 512;
constexpr int kPpOCol = 0, kPpSCol = 256;      // + 128 * tile

template <int NL>
__global__ void __launch_bounds__(kPpThreads, 1)
attn_pingpong_kernel(const __grid_constant__ AttnLayers<NL> layers, const sd_batch bt,
                     const float scale_log2, const AttnPlan plan, int32_t* status) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* q_smem = smem;
    uint8_t* k_smem = smem + kPpQBytes;
    uint8_t* v_smem = k_smem + kPpKStages * kPpStage;
    uint64_t* bars = reinterpret_cast<uint64_t*>(v_smem + kPpVStages * kPpStage);
    uint64_t* k_full = bars;             // [2] TMA -> MMA
    uint64_t* k_empty = bars + 2;        // [2] MMA -> TMA
    uint64_t* v_full = bars + 4;         // [2]
    uint64_t* v_empty = bars + 6;        // [2]
    uint64_t* s_full = bars + 8;         // [2] per row tile: MMA -> softmax (scores of key tile j; phase j)
    uint64_t* p_full = bars + 10;        // [2] per row tile: softmax -> MMA (P written, O rescaled; 4 warps; phase j)
    uint64_t* pv_done = bars + 12;       // [2] per row tile: MMA -> softmax (O updated by key tile j; phase j)
    uint64_t* q_full = bars + 14;        // [2] per row tile: softmax -> MMA (Q staged; 4 warps)
    uint64_t* o_full = bars + 16;        // MMA -> softmax (single use: every MMA of the CTA has completed)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 17);
    int* abort_flag = reinterpret_cast<int*>(bars + 18);
    int* s_seq = reinterpret_cast<int*>(bars + 19);

    // warp index as a value the compiler knows to be warp-uniform, so that role dispatch is uniform
    // control flow (a warp's non-existent lanes do not take part in the shuffle)
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    const int chunk = blockIdx.x;
    const int pair = blockIdx.y;                           // row tiles 2 * pair and 2 * pair + 1
    const bool has_b = (2 * pair + 1) < plan.row_tiles;
    // blockIdx.z enumerates (sequence rank, layer, KV head), longest sequences first in every layer
    const int zz = (int)blockIdx.z + plan.z0;
    const int kvh = zz % bt.Hkv;
    const int lb = zz / bt.Hkv;
    const int rank_b = lb / plan.n_layers;
    int b = rank_b;
    if (plan.ranked) {
        if ((int)threadIdx.x < bt.B) {
            const int mine = __ldg(bt.len + threadIdx.x);
            int r = 0;
            for (int j = 0; j < bt.B; ++j) {
                const int other = __ldg(bt.len + j);
                r += (other > mine || (other == mine && j < (int)threadIdx.x)) ? 1 : 0;
            }
            if (r == rank_b) *s_seq = threadIdx.x;
        }
        __syncthreads();
        b = *s_seq;
    }
    const AttnLayer& ly = layers.l[lb % plan.n_layers];
    const CUtensorMap* const map_kc = &ly.k_cache;
    const CUtensorMap* const map_vc = &ly.v_cache;
    const CUtensorMap* const map_kt = &ly.k_tree;
    const CUtensorMap* const map_vt = &ly.v_tree;
    const uint16_t* __restrict__ q = ly.q;
    __nv_bfloat16* __restrict__ out = ly.out;
    float* __restrict__ lse = ly.lse;
    const int num_blocks = ly.num_blocks;
    const int G = bt.Hq / bt.Hkv;
    const int T = bt.T_max;
    const int n = min(max(bt.n_nodes[b], 0), T);
    const int len = max(bt.len[b], 0);

    // 64-key blocks of this CTA: cache blocks [t0, t1) and, for the last chunk, the tree's block.
    // Chunks hold an even number of blocks, so that only a sequence's very last key tile can be a half.
    int tiles_total = (len + 63) / 64;
    if (tiles_total > bt.max_blocks_per_seq) {             // the block table does not cover this length
        if (threadIdx.x == 0) set_status(status, SD_ERR_BOUNDS);
        tiles_total = bt.max_blocks_per_seq;
    }
    const int tpc = (((tiles_total + plan.n_chunks - 1) / plan.n_chunks) + 1) & ~1;
    const int t0 = min(chunk * tpc, tiles_total);
    const int t1 = min(t0 + tpc, tiles_total);
    const bool has_tree = (chunk == plan.n_chunks - 1);
    const int n_pref = t1 - t0;
    const int hb = n_pref + (has_tree ? 1 : 0);            // blocks
    const int nt = (hb + 1) >> 1;                          // key tiles of up to two blocks
    const bool aligned = (smem_u32(smem) & 1023u) == 0;    // swizzled tiles need 1 KiB alignment
    if (!aligned && threadIdx.x == 0) set_status(status, SD_ERR_UNSUPPORTED);
    // A CTA without key tiles has nothing to compute, but it still takes part in the cluster barriers.
    const bool active = (nt > 0) && aligned;
    const bool clustered = (plan.n_chunks > 1);
    float m_used = -INFINITY, l = 0.f;                     // softmax state of this thread's row (warps 0-7)
    uint32_t tmem_base = 0;
    const long long wait_limit = plan.wait_cycles;

    if (active) {
    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int i = 0; i < 2; ++i) {
            mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1); mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1);
            mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 4); mbar_init(&pv_done[i], 1); mbar_init(&q_full[i], 4);
        }
        mbar_init(o_full, 1);
        fence_barrier_init();
    }
    if (warp == kPpTmaWarp) {                              // a full warp (the MMA warp is a single thread)
        tmem_alloc(tmem_slot, kPpTmemCols);
        tmem_relinquish();
    }
    if (warp == kPpTmaWarp && lane == 0) {
        prefetch_tensormap(map_kc); prefetch_tensormap(map_vc);
        prefetch_tensormap(map_kt); prefetch_tensormap(map_vt);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    tmem_base = *tmem_slot;

    if (warp == kPpTmaWarp) {
        // ------------------------------------------------------------ TMA producer (one thread)
        // K and V tiles travel through separate rings and are issued independently, whichever slot
        // frees first.  A tile is up to two blocks; each block arrives as two 64-wide D-halves.
        if (lane == 0) {
            const uint64_t pol = policy_evict_first();
            const int32_t* table = bt.block_table + (size_t)b * bt.max_blocks_per_seq;
            int jk = 0, jv = 0;
            bool ok = true;
            long long t_last = clock64();
            auto issue = [&](int j, bool is_v) {
                const int s = j & 1;
                uint64_t* full = (is_v ? v_full : k_full) + s;
                uint8_t* dst = (is_v ? v_smem : k_smem) + s * kPpStage;
                const int nk = min(2, hb - 2 * j);
                mbar_arrive_expect_tx(full, (uint32_t)(nk * 2 * kPpBlockHalf));
                for (int u = 0; u < nk; ++u) {
                    const int bi = 2 * j + u;
                    uint8_t* d = dst + u * kPpBlockHalf;
                    if (bi >= n_pref) {
                        const CUtensorMap* m = is_v ? map_vt : map_kt;
                        tma_load_3d(d, m, 0, kvh, b * T, full, pol);
                        tma_load_3d(d + kPpHalf, m, 64, kvh, b * T, full, pol);
                    } else {
                        int blk = __ldg(table + t0 + bi);
                        if (blk < 0 || blk >= num_blocks) { set_status(status, SD_ERR_BOUNDS); blk = 0; }
                        const CUtensorMap* m = is_v ? map_vc : map_kc;
                        const int y = (blk * bt.Hkv + kvh) * 64;
                        tma_load_2d(d, m, 0, y, full, pol);
                        tma_load_2d(d + kPpHalf, m, 64, y, full, pol);
                    }
                }
            };
            while ((jk < nt || jv < nt) && ok) {
                bool progress = false;
                if (jk < nt && mbar_try_wait(&k_empty[jk & 1], ((uint32_t)(jk >> 1) & 1u) ^ 1u)) {
                    issue(jk, false);
                    ++jk;
                    progress = true;
                }
                if (jv < nt && mbar_try_wait(&v_empty[jv & 1], ((uint32_t)(jv >> 1) & 1u) ^ 1u)) {
                    issue(jv, true);
                    ++jv;
                    progress = true;
                }
                if (progress) {
                    t_last = clock64();
                } else if (*reinterpret_cast<volatile int*>(abort_flag) || clock64() - t_last > wait_limit) {
                    *reinterpret_cast<volatile int*>(abort_flag) = 1;
                    ok = false;
                }
            }
            if (!ok) {
                set_status(status, SD_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);      // let copies in flight land
            }
        }
    } else if (warp == kPpMmaWarp) {
        // ------------------------------------------------------------ MMA issuer (a warp of one thread)
        // Issue order per key tile j:  P.V of A | scores of A for tile j + 1 | P.V of B | scores of B
        // for tile j + 1.  The instructions of one thread execute in order, so the next score tile of a
        // row tile may overwrite the columns its P.V has just read, and the softmax of one row tile
        // has the other tile's two MMA groups to hide behind.
        {
            const uint32_t idesc_o = make_idesc_bf16(kRowTile, kD, false, true);          // O += P . V
            const uint32_t idesc_s2 = make_idesc_bf16(kRowTile, 128, false, false);      // S = Q . K^T, 128 keys
            const uint32_t idesc_s1 = make_idesc_bf16(kRowTile, 64, false, false);       // a last tile of one block
            // k-steps only move the (16-byte granular) start-address field in the low bits
            const uint64_t qdesc_base = make_smem_desc(smem_u32(q_smem), 16, 1024, 128);
            const uint64_t kdesc_base = make_smem_desc(smem_u32(k_smem), 16, 1024, 128);
            // V is stored [key][d]: N (= d) contiguous; D-halves kPpHalf apart, 8-key groups 1 KiB apart
            const uint64_t vdesc_base = make_smem_desc(smem_u32(v_smem), kPpHalf, 1024, 128);
            const uint32_t tmem_o = tmem_base + kPpOCol, tmem_s = tmem_base + kPpSCol;
            bool ok = true;
            auto issue_s = [&](int j, int x) {                     // scores of key tile j for row tile x
                const uint64_t kd = kdesc_base + (uint64_t)((j & 1) * (kPpStage >> 4));
                const uint64_t qd = qdesc_base + (uint64_t)(x * (kPpStage >> 4));
                const uint32_t d = tmem_s + x * 128;
                const uint32_t idesc = (hb - 2 * j >= 2) ? idesc_s2 : idesc_s1;
#pragma unroll
                for (int k = 0; k < kD / 16; ++k)
                    mma_ss(d, qd + (uint64_t)((k >> 2) * (kPpHalf >> 4) + (k & 3) * 2),
                           kd + (uint64_t)((k >> 2) * (kPpHalf >> 4) + (k & 3) * 2), idesc, k != 0 ? 1u : 0u);
                mma_commit(&s_full[x]);
            };
            auto issue_pv = [&](int j, int x) {                    // O_x += P_x . V of key tile j
                const uint64_t vd = vdesc_base + (uint64_t)((j & 1) * (kPpStage >> 4));
                const uint32_t pa = tmem_s + x * 128;              // P straight from TMEM: 16 keys = 8 columns
                const uint32_t first = (j != 0) ? 1u : 0u;
                if (hb - 2 * j >= 2) {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        mma_ts(tmem_o + x * 128, pa + k * 8, vd + (uint64_t)(k * (2048 >> 4)), idesc_o, k != 0 ? 1u : first);
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        mma_ts(tmem_o + x * 128, pa + k * 8, vd + (uint64_t)(k * (2048 >> 4)), idesc_o, k != 0 ? 1u : first);
                }
                mma_commit(&pv_done[x]);
            };
            ok = mbar_wait(&q_full[0], 0, abort_flag, wait_limit) && mbar_wait(&k_full[0], 0, abort_flag, wait_limit);
            if (ok) {
                tc_fence_after_sync();
                issue_s(0, 0);
                if (has_b) {
                    ok = mbar_wait(&q_full[1], 0, abort_flag, wait_limit);
                    if (ok) { tc_fence_after_sync(); issue_s(0, 1); }
                }
                mma_commit(&k_empty[0]);
            }
            for (int j = 0; j < nt && ok; ++j) {
                const uint32_t ph = (uint32_t)j & 1u;
                const bool more = (j + 1 < nt);
                if (!mbar_wait(&p_full[0], ph, abort_flag, wait_limit)) { ok = false; break; }
                if (!mbar_wait(&v_full[j & 1], (uint32_t)(j >> 1) & 1u, abort_flag, wait_limit)) { ok = false; break; }
                tc_fence_after_sync();
                issue_pv(j, 0);
                if (more) {
                    if (!mbar_wait(&k_full[(j + 1) & 1], (uint32_t)((j + 1) >> 1) & 1u, abort_flag, wait_limit)) { ok = false; break; }
                    tc_fence_after_sync();
                    issue_s(j + 1, 0);
                }
                if (has_b) {
                    if (!mbar_wait(&p_full[1], ph, abort_flag, wait_limit)) { ok = false; break; }
                    tc_fence_after_sync();
                    issue_pv(j, 1);
                }
                mma_commit(&v_empty[j & 1]);
                if (more) {
                    if (has_b) issue_s(j + 1, 1);
                    mma_commit(&k_empty[(j + 1) & 1]);
                }
            }
            mma_commit(o_full);
            if (!ok) {
                // unwinding: nothing may give tensor memory back while an MMA issued above still runs
                set_status(status, SD_ERR_TIMEOUT);
                mbar_wait_plain(o_full, 0, wait_limit);
            }
        }
    } else {
        // ------------------------------------------------------------ softmax: one thread per row
        const int x = warp >> 2;                           // row tile of this warp: 0 = A, 1 = B
        const int wq = warp & 3;                           // TMEM lane quadrant
        const int tid = wq * 32 + lane;                    // row within the tile
        const int rt = 2 * pair + x;
        const int row = rt * kRowTile + tid;
        const int node = row / G;
        const int g = row - node * G;
        const bool row_ok = (row < plan.rows) && (node < n);
        const bool tile_on = (x == 0) || has_b;
        const bool warp_live = __any_sync(0xffffffffu, row_ok);     // a warp of padding rows only skips the arithmetic
        bool ok = true;
        if (tile_on) {
            {   // stage this row of Q (zeros for padding rows) in the swizzled K-major layout
                const uint4* src = reinterpret_cast<const uint4*>(
                    q + (((size_t)b * T + (row_ok ? node : 0)) * bt.Hq + kvh * G + (row_ok ? g : 0)) * kD);
                uint8_t* qx = q_smem + x * kPpStage;
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    uint4 u = row_ok ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
                    *reinterpret_cast<uint4*>(qx + (c >> 3) * kPpHalf + tid * 128 + (((c & 7) ^ (tid & 7)) << 4)) = u;
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&q_full[x]);
            }
            const uint64_t amask = row_ok ? bt.anc_mask[(size_t)b * T + node] : ~0ull;
            const uint32_t lane_field = (uint32_t)(wq * 32) << 16;
            const uint32_t tmem_ox = tmem_base + lane_field + kPpOCol + x * 128;
            const uint32_t tmem_sx = tmem_base + lane_field + kPpSCol + x * 128;
            for (int j = 0; j < nt && ok; ++j) {
                const uint32_t ph = (uint32_t)j & 1u;
                const int nk = min(2, hb - 2 * j);
                if (!mbar_wait(&s_full[x], ph, abort_flag, wait_limit)) { ok = false; break; }
                tc_fence_after_sync();
                // Keys that no row may see (cache slots at and beyond len, rows of unused tree nodes) carry
                // weight 0, but 0 x NaN or 0 x Inf would still poison the accumulator: the threads of row
                // tile A (thread <-> key row of the tile) clear those V rows in shared memory before P.V reads
                // them; the arrival on p_full below orders the two, and P.V of B is issued behind P.V of A.
                // This comes after the wait for the scores of tile j: they were issued behind P.V of tile
                // j - 1, which waited for its own V tile, so the slot's barrier is by now in the phase of
                // tile j and the parity wait below cannot be taken for an earlier phase.
                if (x == 0) {
                    const int u = tid >> 6, r = tid & 63;
                    const int bi = 2 * j + u;
                    const int my_rows = (bi >= n_pref) ? n : min(64, len - (t0 + bi) * 64);
                    const bool need = (u < nk) && (r >= my_rows);
                    if (__any_sync(0xffffffffu, need)) {
                        if (!mbar_wait(&v_full[j & 1], (uint32_t)(j >> 1) & 1u, abort_flag, wait_limit)) { ok = false; break; }
                        if (need) {
                            uint4* z = reinterpret_cast<uint4*>(v_smem + (j & 1) * kPpStage + tid * 128);
#pragma unroll
                            for (int c = 0; c < 8; ++c) {
                                z[c] = make_uint4(0, 0, 0, 0);
                                z[c + kPpHalf / 16] = make_uint4(0, 0, 0, 0);
                            }
                            fence_proxy_async_smem();
                        }
                    }
                }
                if (warp_live) {
                    for (int u = 0; u < nk && ok; ++u) {
                        // one block of 64 keys: scores in columns 64u.., probabilities go to columns 32u..
                        const int bi = 2 * j + u;
                        const bool tree = (bi >= n_pref);
                        const int valid = tree ? 64 : len - (t0 + bi) * 64;   // keys of this block inside the prefix
                        // The scores arrive in two halves; the second half is in flight while the first is
                        // processed.  Raw scores stay unscaled: scale * log2(e) is folded into the exponent's FMA.
                        uint32_t r0[32], r1[32];
                        tmem_ld32(tmem_sx + u * 64, r0);
                        tmem_ld_wait();
                        tmem_ld32(tmem_sx + u * 64 + 32, r1);
                        const uint32_t mask_lo = tree ? (uint32_t)amask : (valid >= 32 ? ~0u : ((1u << max(valid, 0)) - 1u));
                        const uint32_t mask_hi = tree ? (uint32_t)(amask >> 32)
                                                      : (valid >= 64 ? ~0u : (valid <= 32 ? 0u : ((1u << (valid - 32)) - 1u)));
                        const bool masked = tree || valid < 64;
                        if (masked) {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                r0[c] = ((mask_lo >> c) & 1u) ? r0[c] : 0xff800000u;      // -inf
                        }
                        // The exponentials are taken against the current reference maximum right away, while the
                        // block's own maximum is found alongside (independent instruction streams); only when that
                        // maximum turns out to exceed the reference by more than the threshold (rare after the
                        // first tiles) is the reference raised and the block's exponentials redone.
                        uint32_t pk[32];
                        float ps[4] = {0.f, 0.f, 0.f, 0.f};
                        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                        const float neg_m = -m_used;
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const float a = __uint_as_float(r0[2 * c]), bq = __uint_as_float(r0[2 * c + 1]);
                            mx[c & 3] = max3(mx[c & 3], a, bq);
                            const float p0 = ex2_approx(fmaf(a, scale_log2, neg_m));
                            const float p1 = ex2_approx(fmaf(bq, scale_log2, neg_m));
                            ps[c & 3] += p0 + p1;
                            __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                            pk[c] = *reinterpret_cast<uint32_t*>(&h);
                        }
                        tmem_ld_wait();
                        if (masked) {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                r1[c] = ((mask_hi >> c) & 1u) ? r1[c] : 0xff800000u;
                        }
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const float a = __uint_as_float(r1[2 * c]), bq = __uint_as_float(r1[2 * c + 1]);
                            mx[c & 3] = max3(mx[c & 3], a, bq);
                            const float p0 = ex2_approx(fmaf(a, scale_log2, neg_m));
                            const float p1 = ex2_approx(fmaf(bq, scale_log2, neg_m));
                            ps[c & 3] += p0 + p1;
                            __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                            pk[16 + c] = *reinterpret_cast<uint32_t*>(&h);
                        }
                        const float mt = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2;   // scale > 0
                        // raise the reference maximum only when it would grow by more than the threshold
                        // (always on the first block: m_used = -inf)
                        const bool raise = mt > m_used + kRescaleThreshold;
                        if (__any_sync(0xffffffffu, raise)) {
                            const float alpha = raise ? exp2f(m_used - mt) : 1.f;    // 0 on the first block
                            if (j > 0) {
                                // everything accumulated so far was taken against the old reference
                                if (!mbar_wait(&pv_done[x], (uint32_t)(j - 1) & 1u, abort_flag, wait_limit)) { ok = false; break; }
                                tc_fence_after_sync();
#pragma unroll
                                for (int cc = 0; cc < 4; ++cc) {
                                    uint32_t o[32];
                                    tmem_ld32(tmem_ox + cc * 32, o);
                                    tmem_ld_wait();
#pragma unroll
                                    for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                                    tmem_st32(tmem_ox + cc * 32, o);
                                }
                            }
                            if (u > 0) {
                                // so were the probabilities of this tile's first block, already in TMEM
                                uint32_t p0[32];
                                tmem_st_wait();
                                tmem_ld32(tmem_sx, p0);
                                tmem_ld_wait();
#pragma unroll
                                for (int c = 0; c < 32; ++c) {
                                    __nv_bfloat162 h = __floats2bfloat162_rn(bf16lo(p0[c]) * alpha, bf16hi(p0[c]) * alpha);
                                    p0[c] = *reinterpret_cast<uint32_t*>(&h);
                                }
                                tmem_st32(tmem_sx, p0);
                            }
                            tmem_st_wait();
                            l *= alpha;
                            if (raise) m_used = mt;
                            // redo the block against the new reference (same values for rows that did not raise)
                            const float neg_m2 = -m_used;
                            ps[0] = ps[1] = ps[2] = ps[3] = 0.f;
#pragma unroll
                            for (int c = 0; c < 16; ++c) {
                                const float p0 = ex2_approx(fmaf(__uint_as_float(r0[2 * c]), scale_log2, neg_m2));
                                const float p1 = ex2_approx(fmaf(__uint_as_float(r0[2 * c + 1]), scale_log2, neg_m2));
                                const float p2 = ex2_approx(fmaf(__uint_as_float(r1[2 * c]), scale_log2, neg_m2));
                                const float p3 = ex2_approx(fmaf(__uint_as_float(r1[2 * c + 1]), scale_log2, neg_m2));
                                ps[c & 3] += (p0 + p1) + (p2 + p3);
                                __nv_bfloat162 h0 = __floats2bfloat162_rn(p0, p1);
                                __nv_bfloat162 h1 = __floats2bfloat162_rn(p2, p3);
                                pk[c] = *reinterpret_cast<uint32_t*>(&h0);
                                pk[16 + c] = *reinterpret_cast<uint32_t*>(&h1);
                            }
                        }
                        l += (ps[0] + ps[1]) + (ps[2] + ps[3]);
                        // P replaces score columns this thread has already consumed (its own TMEM lane)
                        tmem_st32(tmem_sx + u * 32, pk);
                    }
                    tmem_st_wait();
                }
                if (!ok) break;
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0 && !(plan.withhold && j == 0)) mbar_arrive(&p_full[x]);
            }
            // ------------------------------------------------------------ epilogue
            if (ok) ok = mbar_wait(o_full, 0, abort_flag, wait_limit);
            if (ok && !clustered) {
                // single chunk: normalise and write bf16 output
                tc_fence_after_sync();
                const size_t orow = ((size_t)b * T + node) * bt.Hq + kvh * G + g;
                const float inv = 1.f / l;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t o[32];
                    if (warp_live) {
                        tmem_ld32(tmem_ox + cc * 32, o);
                        tmem_ld_wait();
                    }
                    if (row < plan.rows) {
                        uint32_t w[16];
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const float a = row_ok ? __uint_as_float(o[2 * c]) * inv : 0.f;
                            const float bb = row_ok ? __uint_as_float(o[2 * c + 1]) * inv : 0.f;
                            __nv_bfloat162 hh = __floats2bfloat162_rn(a, bb);
                            w[c] = *reinterpret_cast<uint32_t*>(&hh);
                        }
                        uint4* dst = reinterpret_cast<uint4*>(out + orow * kD + cc * 32);
#pragma unroll
                        for (int c = 0; c < 4; ++c) dst[c] = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
                    }
                }
                if (row < plan.rows && lse) lse[orow] = row_ok ? (m_used + log2f(l)) * 0.6931471805599453f : 0.f;
            } else if (ok) {
                // several chunks: park (m, l, unnormalised O) in this CTA's own shared memory, where the
                // CTAs of the cluster read it: O of tile A in the K ring, of tile B in the V ring (idle by
                // now: every MMA has completed), the statistics in the Q area.  16-byte pieces of a row are
                // XOR-swizzled by the row index so that the per-row accesses of a warp spread over the banks.
                tc_fence_after_sync();
                float* xo = reinterpret_cast<float*>(x == 0 ? k_smem : v_smem);
                float* xs = reinterpret_cast<float*>(q_smem + x * kPpStage);
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t o[32];
                    if (warp_live) {
                        tmem_ld32(tmem_ox + cc * 32, o);
                        tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int c = 0; c < 32; ++c) o[c] = 0u;
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        *reinterpret_cast<uint4*>(xo + tid * kD + (((cc * 8 + k) ^ (tid & 31)) << 2)) =
                            make_uint4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
                }
                xs[tid] = warp_live ? m_used : -INFINITY;
                xs[kRowTile + tid] = warp_live ? l : 0.f;
            } else if (lane == 0) {
                set_status(status, SD_ERR_TIMEOUT);
            }
        }
    }
    }   // active

    if (clustered) {
        // every thread of every CTA of the cluster: exchange areas are complete and visible
        __syncwarp();
        cluster_arrive_release();
        cluster_wait_acquire();
        if (warp < 8 && (warp < 4 || has_b)) {
            const int x = warp >> 2;
            const uint32_t xo_addr = smem_u32(x == 0 ? k_smem : v_smem);
            const uint32_t xs_addr = smem_u32(q_smem + x * kPpStage);
            const MergeCtx mc{bt, plan, out, lse, xo_addr, xs_addr,
                              chunk, 2 * pair + x, b, kvh, n, tpc, tiles_total, warp & 3, lane};
            if (plan.n_chunks == 2) merge_rows<2>(mc);
            else if (plan.n_chunks == 4) merge_rows<4>(mc);
            else merge_rows<8>(mc);
        }
        // every CTA keeps its shared memory alive until all the others have read it
        __syncwarp();
        cluster_arrive_release();
        cluster_wait_acquire();
    }
    if (!active) return;
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kPpTmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kPpTmemCols);
    }
}

template <int NL>
sd_status launch_rows2(const AttnLayers<NL>& layers, const sd_batch& bt, float scale, const AttnPlan& plan,
                       int z_count, int32_t* dev_status, cudaStream_t st) {
    auto kern = attn_pingpong_kernel<NL>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kPpSmem) != cudaSuccess)
        return SD_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.n_chunks, plan.ctas_per_group, z_count);
    cfg.blockDim = dim3(kPpThreads);
    cfg.dynamicSmemBytes = kPpSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;      // the key chunks of one pair of row tiles form a cluster
    attr[0].val.clusterDim.x = plan.n_chunks;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, layers, bt, scale * kLog2e, plan, dev_status) != cudaSuccess)
        return SD_ERR_CUDA;
    return SD_OK;
}
template sd_status launch_rows2<1>(const AttnLayers<1>&, const sd_batch&, float, const AttnPlan&, int, int32_t*,
                                   cudaStream_t);
template sd_status launch_rows2<kMaxLayersPerLaunch>(const AttnLayers<kMaxLayersPerLaunch>&, const sd_batch&, float,
                                                     const AttnPlan&, int, int32_t*, cudaStream_t);

}  // namespace sdv
