// Tree-masked GQA attention over a paged prefix cache plus the tree's own KV,
// on the 5th-generation tensor cores (tcgen05 + TMEM), split-KV.
//
// All T*G query rows that share one KV head (node-major: row = node*G + g) are
// processed against every K/V byte exactly once per 128-row tile: with 60 nodes
// and 7 grouped heads that is 420 rows per K/V row, which makes the step
// compute-bound, so both S = Q.K^T and O += P.V run as tcgen05.mma with
// accumulators in TMEM.
//
// One CTA = (sequence, KV head, 128-row tile, key chunk).  Its key tiles are the
// 64-token cache blocks of the chunk (TMA, 128-byte swizzle, located through the
// block table) and, for the last chunk, one extra tile holding the tree's own
// keys, masked per row by the node's ancestor bitmask.  Softmax runs one thread
// per row straight out of TMEM (no cross-thread reductions); the running maximum
// is only raised when it grows by more than 2^8, so the accumulator in TMEM is
// rescaled rarely.  P goes back into TMEM and feeds the second MMA from there.
// With one chunk the CTA writes the output itself; otherwise the chunks of a row
// tile form a thread-block cluster: every CTA pushes its (max, sum, unnormalised
// O) rows into the shared memory of the CTA that finishes them (remote stores),
// and each CTA merges its share of the rows locally, in chunk order.
// The launch is a programmatic dependent launch: barriers, tensor memory and
// tensor-map prefetch are set up before the kernel waits for the kernel ahead of
// it in the stream, so consecutive per-layer calls overlap their ends.
#include "attention_shared.cuh"

namespace sdv {

constexpr int kKeyTile = 64;                   // keys per tile = one cache block
constexpr int kAttThreads = 161;               // warps 0-3 softmax, warp 4 TMA, warp 5 = ONE thread: MMA issuer
constexpr int kTmaWarp = 4, kMmaWarp = 5;
constexpr int kSubTile = kKeyTile * 128;       // bytes of a [64][64] bf16 swizzled sub-tile (8 KiB)
constexpr int kQBytes = 2 * kRowTile * 128;    // Q tile: two D-halves of [128][64] bf16 (32 KiB)
constexpr int kKVStage = 2 * kSubTile;         // one K (or V) tile: two D-halves (16 KiB)
constexpr int kKStages = 3;                    // K tiles are consumed a tile ahead of V
constexpr int kVStages = 2;
constexpr int kAttSmem = kQBytes + (kKStages + kVStages) * kKVStage + 256;
constexpr int kTmemCols = 256;                 // O: 0..127, S/P buffers: 128..191, 192..255
// P (bf16, two keys per 32-bit column) overwrites the first 32 columns of the S buffer it came from

template <int NL>
__global__ void __launch_bounds__(kAttThreads, 2)
attn_umma_kernel(const __grid_constant__ AttnLayers<NL> layers, const sd_batch bt,
                 const float scale_log2, const AttnPlan plan, int32_t* status) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* q_smem = smem;
    uint8_t* k_smem = smem + kQBytes;
    uint8_t* v_smem = k_smem + kKStages * kKVStage;
    uint64_t* bars = reinterpret_cast<uint64_t*>(v_smem + kVStages * kKVStage);
    uint64_t* k_full = bars;             // [3] TMA -> MMA
    uint64_t* k_empty = bars + 3;        // [3] MMA -> TMA
    uint64_t* v_full = bars + 6;         // [2]
    uint64_t* v_empty = bars + 8;        // [2]
    uint64_t* s_full = bars + 10;        // [2] MMA -> softmax (scores of tile j in buffer j&1)
    uint64_t* p_full = bars + 12;        // [2] softmax -> MMA (P written into buffer j&1, O rescaled); one
                                         //     barrier per buffer so that a warp running a tile ahead
                                         //     cannot complete the previous tile's phase
    uint64_t* pv_done = bars + 14;       // MMA -> softmax   (O updated by tile j; phase j)
    uint64_t* o_full = bars + 15;        // MMA -> softmax   (single use: every MMA of the CTA has completed)
    uint64_t* q_full = bars + 16;        // softmax -> MMA   (Q staged)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 17);
    int* abort_flag = reinterpret_cast<int*>(bars + 18);

    // warp index as a value the compiler knows to be warp-uniform, so that role dispatch is uniform
    // control flow (a warp's non-existent lanes do not take part in the shuffle)
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    const int chunk = blockIdx.x;
    const int rt = blockIdx.y;
    // blockIdx.z enumerates (sequence rank, layer, KV head): the CTAs of the longest sequences are
    // dispatched first, in every layer, so that a ragged batch does not end on a few long stragglers.
    // The rank -> sequence lookup is done here (up to 64 sequences: each of the first B threads ranks
    // one sequence by cached length, ties by index); larger batches, and launches that fit the GPU in
    // one wave, run in index order.
    const int zz = (int)blockIdx.z + plan.z0;
    const int kvh = zz % bt.Hkv;
    const int lb = zz / bt.Hkv;
    const int rank_b = lb / plan.n_layers;
    const AttnLayer& ly = layers.l[lb % plan.n_layers];
    const CUtensorMap* const map_kc = &ly.k_cache;
    const CUtensorMap* const map_vc = &ly.v_cache;
    const CUtensorMap* const map_kt = &ly.k_tree;
    const CUtensorMap* const map_vt = &ly.v_tree;

    // Set-up that touches no global memory comes first: when the launch is allowed to start before the
    // kernel ahead of it in the stream has finished (programmatic dependent launch: one attention call
    // per layer, back to back), it overlaps that kernel's tail.  The kernel behind this one may start
    // its own set-up as soon as every CTA of this grid is running.
    griddep_launch_dependents();
    const bool aligned = (smem_u32(smem) & 1023u) == 0;    // swizzled tiles need 1 KiB alignment
    uint32_t tmem_base = 0;
    if (aligned) {
        if (warp == kMmaWarp) {                            // (a thread with nothing else to do at this point)
            *abort_flag = 0;
            for (int i = 0; i < kKStages; ++i) { mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1); }
            for (int i = 0; i < kVStages; ++i) { mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1); }
            for (int i = 0; i < 2; ++i) { mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 4); }
            mbar_init(pv_done, 1); mbar_init(q_full, 4); mbar_init(o_full, 1);
            fence_barrier_init();
        }
        if (warp == kTmaWarp) {                            // a full warp (the MMA warp is a single thread)
            tmem_alloc(tmem_slot, kTmemCols);
            tmem_relinquish();
        }
        if (warp == kTmaWarp && lane == 0) {
            prefetch_tensormap(map_kc); prefetch_tensormap(map_vc);
            prefetch_tensormap(map_kt); prefetch_tensormap(map_vt);
        }
    } else if (threadIdx.x == 0) {
        set_status(status, SD_ERR_UNSUPPORTED);
    }
    // everything below reads (or writes) global memory that the kernel ahead may still be working on
    griddep_wait();

    int b = rank_b;
    if (plan.ranked) {
        // (the slot lives in the dynamic shared-memory block: a static variable would push that block's
        //  1 KiB-aligned start and cost the second resident CTA)
        int& s_seq = *reinterpret_cast<int*>(bars + 19);
        if ((int)threadIdx.x < bt.B) {
            const int mine = __ldg(bt.len + threadIdx.x);
            int r = 0;
            for (int j = 0; j < bt.B; ++j) {
                const int other = __ldg(bt.len + j);
                r += (other > mine || (other == mine && j < (int)threadIdx.x)) ? 1 : 0;
            }
            if (r == rank_b) s_seq = threadIdx.x;
        }
        __syncthreads();
        b = s_seq;
    }
    const uint16_t* __restrict__ q = ly.q;
    __nv_bfloat16* __restrict__ out = ly.out;
    float* __restrict__ lse = ly.lse;
    const int num_blocks = ly.num_blocks;
    const int G = bt.Hq / bt.Hkv;
    const int T = bt.T_max;
    // A last row tile of at most 64 rows (420 rows = 3 x 128 + 36) runs its MMAs with M = 64: the
    // accumulator rows then sit in lanes 0..15 of each 32-lane TMEM quadrant (row = 16 * quadrant + lane),
    // the tensor cores work at half width and only 64 rows of Q are staged and re-read per key tile.
    const bool m64 = (plan.rows - rt * kRowTile) <= 64;
    // The softmax threads request their row of Q together with the lengths, before anything waits for
    // either.  A node index below T_max always addresses memory of q; rows of unused nodes are replaced
    // by zeros when staged.
    const int q_tid = warp * 32 + lane;
    const int q_row_in_tile = (warp >= 4) ? -1 : (m64 ? (lane < 16 ? warp * 16 + lane : -1) : q_tid);   // -1: no row
    const int q_row = (q_row_in_tile >= 0) ? rt * kRowTile + q_row_in_tile : plan.rows;
    const int n = min(max(__ldg(bt.n_nodes + b), 0), T);      // (requested before the row, needed before it)
    const int len = max(__ldg(bt.len + b), 0);
    uint4 q_regs[16];
    if (q_row < plan.rows) {
        const int node = q_row / G;
        const uint4* src = reinterpret_cast<const uint4*>(
            q + (((size_t)b * T + node) * bt.Hq + kvh * G + (q_row - node * G)) * kD);
#pragma unroll
        for (int c = 0; c < 16; ++c) q_regs[c] = __ldg(src + c);
    }

    // key tiles of this CTA: cache blocks [t0, t1) and, for the last chunk, the tree tile
    int tiles_total = (len + kKeyTile - 1) / kKeyTile;
    if (tiles_total > bt.max_blocks_per_seq) {             // the block table does not cover this length
        if (threadIdx.x == 0) set_status(status, SD_ERR_BOUNDS);
        tiles_total = bt.max_blocks_per_seq;
    }
    const int tpc = (tiles_total + plan.n_chunks - 1) / plan.n_chunks;
    const int t0 = min(chunk * tpc, tiles_total);
    const int t1 = min(t0 + tpc, tiles_total);
    const bool has_tree = (chunk == plan.n_chunks - 1);
    const int nt = (t1 - t0) + (has_tree ? 1 : 0);
    // A CTA without key tiles has nothing to compute, but it still takes part in the cluster barriers.
    const bool active = (nt > 0) && aligned;
    const bool clustered = (plan.n_chunks > 1);            // cluster = the chunks of one (b, kvh, row tile)
    float m_used = -INFINITY, l = 0.f;                     // softmax state of this thread's row (warps 0-3)
    bool rows_ready = false;                               // ... and whether it completed (clustered launches)

    // the set-up at the top (barriers, tensor memory) is visible to every thread from here on
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (aligned) tmem_base = *tmem_slot;
    const uint32_t tmem_o = tmem_base;
    const uint32_t tmem_s = tmem_base + 128;

    if (active) {
    if (warp == kTmaWarp) {
        // ------------------------------------------------------------ TMA producer (one thread)
        // K and V tiles travel through separate rings and are issued independently, whichever slot
        // frees first: the next K tile (needed early, for the score MMA issued one tile ahead) must
        // not queue behind a V slot that is only released when P.V has finished.
        if (lane == 0) {
            const uint64_t pol = policy_evict_first();
            const int32_t* table = bt.block_table + (size_t)b * bt.max_blocks_per_seq;
            const int n_pref = t1 - t0;
            int jk = 0, jv = 0;
            int blk_k = (n_pref > 0) ? __ldg(table + t0) : 0;      // looked up one tile ahead
            int blk_v = blk_k;
            bool ok = true;
            long long t_last = clock64();
            auto issue = [&](int j, int blk, bool is_v) {
                const int stages = is_v ? kVStages : kKStages;
                const int s = j % stages;
                uint64_t* full = (is_v ? v_full : k_full) + s;
                uint8_t* dst = (is_v ? v_smem : k_smem) + s * kKVStage;
                mbar_arrive_expect_tx(full, kKVStage);
                if (j >= n_pref) {
                    const CUtensorMap* m = is_v ? map_vt : map_kt;
                    tma_load_3d(dst, m, 0, kvh, b * T, full, pol);
                    tma_load_3d(dst + kSubTile, m, 64, kvh, b * T, full, pol);
                } else {
                    if (blk < 0 || blk >= num_blocks) { set_status(status, SD_ERR_BOUNDS); blk = 0; }
                    const CUtensorMap* m = is_v ? map_vc : map_kc;
                    const int y = (blk * bt.Hkv + kvh) * kKeyTile;
                    tma_load_2d(dst, m, 0, y, full, pol);
                    tma_load_2d(dst + kSubTile, m, 64, y, full, pol);
                }
            };
            while ((jk < nt || jv < nt) && ok) {
                bool progress = false;
                if (jk < nt && mbar_try_wait(&k_empty[jk % kKStages], ((uint32_t)(jk / kKStages) & 1u) ^ 1u)) {
                    issue(jk, blk_k, false);
                    ++jk;
                    if (jk < n_pref) blk_k = __ldg(table + t0 + jk);
                    progress = true;
                }
                if (jv < nt && mbar_try_wait(&v_empty[jv % kVStages], ((uint32_t)(jv / kVStages) & 1u) ^ 1u)) {
                    issue(jv, blk_v, true);
                    ++jv;
                    if (jv < n_pref) blk_v = __ldg(table + t0 + jv);
                    progress = true;
                }
                if (progress) {
                    t_last = clock64();
                } else if (*reinterpret_cast<volatile int*>(abort_flag) || clock64() - t_last > plan.wait_cycles) {
                    *reinterpret_cast<volatile int*>(abort_flag) = 1;
                    ok = false;
                }
            }
            if (!ok) {
                set_status(status, SD_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);      // let copies in flight land
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------ MMA issuer
        // This warp consists of one thread (the block has 5 * 32 + 1 threads), so everything in
        // here is uniform control flow on warp-uniform values: tcgen05.mma takes its descriptors
        // from uniform registers, and inside a divergent "lane 0 only" region of a full warp every
        // descriptor would first have to be moved there, instruction by instruction.
        {
            const uint32_t idesc_s = make_idesc_bf16(m64 ? 64 : kRowTile, kKeyTile, false, false);   // S = Q . K^T
            const uint32_t idesc_o = make_idesc_bf16(m64 ? 64 : kRowTile, kD, false, true);          // O += P . V
            // k-steps only move the (16-byte granular) start-address field in the low bits
            const uint64_t qdesc_base = make_smem_desc(smem_u32(q_smem), 16, 1024, 128);
            const uint64_t kdesc_base = make_smem_desc(smem_u32(k_smem), 16, 1024, 128);
            // V is stored [key][d]: N (= d) contiguous; D-halves kSubTile apart, 8-key groups 1 KiB apart
            const uint64_t vdesc_base = make_smem_desc(smem_u32(v_smem), kSubTile, 1024, 128);
            bool ok = mbar_wait(q_full, 0, abort_flag, plan.wait_cycles);
            auto issue_s = [&](int j) -> bool {
                const int s = j & 1;                               // score buffer
                const int ks = j % kKStages;                       // K ring slot
                if (!mbar_wait(&k_full[ks], (uint32_t)(j / kKStages) & 1u, abort_flag, plan.wait_cycles)) return false;
                tc_fence_after_sync();
                const uint64_t kd = kdesc_base + (uint64_t)(ks * (kKVStage >> 4));
                const uint32_t d = tmem_s + s * kKeyTile;
#pragma unroll
                for (int k = 0; k < kD / 16; ++k)
                    mma_ss(d, qdesc_base + (uint64_t)((k >> 2) * ((kRowTile * 128) >> 4) + (k & 3) * 2),
                           kd + (uint64_t)((k >> 2) * (kSubTile >> 4) + (k & 3) * 2), idesc_s, k != 0 ? 1u : 0u);
                mma_commit(&k_empty[ks]);
                mma_commit(&s_full[s]);
                return true;
            };
            if (ok) ok = issue_s(0);
            for (int j = 0; j < nt && ok; ++j) {
                if (j + 1 < nt) ok = issue_s(j + 1);
                if (!ok) break;
                const int s = j & 1;
                const uint32_t ph = (uint32_t)(j >> 1) & 1u;
                if (!mbar_wait(&p_full[s], ph, abort_flag, plan.wait_cycles)) { ok = false; break; }
                const int vs = j % kVStages;
                if (!mbar_wait(&v_full[vs], (uint32_t)(j / kVStages) & 1u, abort_flag, plan.wait_cycles)) { ok = false; break; }
                tc_fence_after_sync();
                const uint64_t vd = vdesc_base + (uint64_t)(vs * (kKVStage >> 4));
                const uint32_t pa = tmem_s + s * kKeyTile;        // P comes straight from TMEM: 16 keys = 8 columns
                const uint32_t first = (j != 0) ? 1u : 0u;
#pragma unroll
                for (int k = 0; k < kKeyTile / 16; ++k)
                    mma_ts(tmem_o, pa + k * 8, vd + (uint64_t)(k * (2048 >> 4)), idesc_o, k != 0 ? 1u : first);
                mma_commit(&v_empty[vs]);
                mma_commit(pv_done);
            }
            mma_commit(o_full);
            if (!ok) {
                // unwinding: nothing may give tensor memory back while an MMA issued above still runs
                set_status(status, SD_ERR_TIMEOUT);
                mbar_wait_plain(o_full, 0, plan.wait_cycles);
            }
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------ softmax: one thread per row
        const int tid = warp * 32 + lane;
        const int row_in_tile = m64 ? (lane < 16 ? warp * 16 + lane : -1) : tid;   // -1: a TMEM lane without a row
        const int row = (row_in_tile >= 0) ? rt * kRowTile + row_in_tile : plan.rows;
        const int node = row / G;
        const int g = row - node * G;
        const bool row_ok = (row < plan.rows) && (node < n);
        {   // stage this row of Q (zeros for padding rows) in the swizzled K-major layout
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                uint4 u = row_ok ? q_regs[c] : make_uint4(0, 0, 0, 0);
                uint8_t* dst = q_smem + (c >> 3) * (kRowTile * 128) + row_in_tile * 128 + (((c & 7) ^ (row_in_tile & 7)) << 4);
                if (row_in_tile >= 0) *reinterpret_cast<uint4*>(dst) = u;
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(q_full);
        }
        const uint64_t amask = row_ok ? bt.anc_mask[(size_t)b * T + node] : ~0ull;
        const uint32_t lane_field = (uint32_t)(warp * 32) << 16;
        bool ok = true;
        for (int j = 0; j < nt && ok; ++j) {
            const int s = j & 1;
            const uint32_t ph = (uint32_t)(j >> 1) & 1u;
            const bool tree = (j >= t1 - t0);
            const int valid = tree ? kKeyTile : len - (t0 + j) * kKeyTile;   // keys of this block inside the prefix
            if (!mbar_wait(&s_full[s], ph, abort_flag, plan.wait_cycles)) { ok = false; break; }
            tc_fence_after_sync();
            // Keys that no row may see (cache slots at and beyond len, rows of unused tree nodes) carry
            // weight 0, but 0 x NaN or 0 x Inf would still poison the accumulator: their V rows are
            // cleared in shared memory before P.V reads them (the arrival on p_full below orders the
            // two), so those slots may hold any bit pattern.  This comes after the wait for the scores
            // of tile j: they were issued behind P.V of tile j - 2, which read the V tile that used this
            // ring slot before, so the slot's barrier is by now in the phase of tile j and the parity
            // wait below cannot be taken for an earlier phase.  A key row is 128 contiguous bytes in each
            // of the two D-halves (the swizzle stays inside a row).
            const int v_rows = tree ? n : valid;
            if (v_rows < kKeyTile && warp < 2) {                     // threads 0..63 <-> key rows
                const int vs = j % kVStages;
                if (!mbar_wait(&v_full[vs], (uint32_t)(j / kVStages) & 1u, abort_flag, plan.wait_cycles)) { ok = false; break; }
                if (tid >= v_rows) {
                    uint4* z = reinterpret_cast<uint4*>(v_smem + vs * kKVStage + tid * 128);
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        z[c] = make_uint4(0, 0, 0, 0);
                        z[c + kSubTile / 16] = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async_smem();
                }
            }
            // The scores arrive in two halves; the second half is in flight while the first is
            // processed.  Raw scores stay unscaled: scale * log2(e) is folded into the exponent's FMA.
            uint32_t r0[32], r1[32];
            tmem_ld32(tmem_s + lane_field + s * kKeyTile, r0);
            tmem_ld_wait();
            tmem_ld32(tmem_s + lane_field + s * kKeyTile + 32, r1);
            const uint32_t mask_lo = tree ? (uint32_t)amask : (valid >= 32 ? ~0u : ((1u << max(valid, 0)) - 1u));
            const uint32_t mask_hi = tree ? (uint32_t)(amask >> 32)
                                          : (valid >= 64 ? ~0u : (valid <= 32 ? 0u : ((1u << (valid - 32)) - 1u)));
            const bool masked = tree || valid < kKeyTile;
            if (masked) {
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    r0[c] = ((mask_lo >> c) & 1u) ? r0[c] : 0xff800000u;      // -inf
            }
            // The exponentials are taken against the current reference maximum right away, while the
            // tile's own maximum is found alongside (independent instruction streams); only when that
            // maximum turns out to exceed the reference by more than the threshold (rare after the
            // first tiles) is the reference raised and the tile's exponentials redone.
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
            // true on the first tile (m_used = -inf); lanes without a row hold stale scores and never ask
            const bool raise = (row_in_tile >= 0) && (mt > m_used + kRescaleThreshold);
            if (__any_sync(0xffffffffu, raise)) {
                if (j > 0) {
                    if (!mbar_wait(pv_done, (uint32_t)(j - 1) & 1u, abort_flag, plan.wait_cycles)) { ok = false; break; }
                    tc_fence_after_sync();
                    const float alpha = raise ? exp2f(m_used - mt) : 1.f;
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t o[32];
                        tmem_ld32(tmem_o + lane_field + cc * 32, o);
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                        tmem_st32(tmem_o + lane_field + cc * 32, o);
                    }
                    tmem_st_wait();
                    l *= alpha;
                }
                if (raise) m_used = mt;
                // redo the tile against the new reference (same values for rows that did not raise)
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
            const float psum = (ps[0] + ps[1]) + (ps[2] + ps[3]);
            l += psum;
            // P replaces the S columns this thread has just consumed (its own TMEM lane)
            tmem_st32(tmem_s + lane_field + s * kKeyTile, pk);
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0 && !(plan.withhold && j == 0)) mbar_arrive(&p_full[s]);
        }
        // ------------------------------------------------------------ epilogue
        // (a parity wait on pv_done would be ambiguous here: the softmax may be two phases ahead of it)
        if (ok) ok = mbar_wait(o_full, 0, abort_flag, plan.wait_cycles);
        if (ok && !clustered) {
            // single chunk: normalise and write bf16 output
            tc_fence_after_sync();
            const int h = kvh * G + g;
            const size_t orow = ((size_t)b * T + node) * bt.Hq + h;
            const float inv = 1.f / l;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                uint32_t o[32];
                tmem_ld32(tmem_o + lane_field + cc * 32, o);
                tmem_ld_wait();
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
            rows_ready = true;         // several chunks: the rows leave for their finishing CTAs below
        } else if (!ok && lane == 0) {
            set_status(status, SD_ERR_TIMEOUT);
        }
    }
    }   // active

    if (clustered) {
        // every thread of every CTA of the cluster: all MMAs and copies of the cluster have completed, so
        // every CTA's K/V rings are free to receive rows
        __syncwarp();
        cluster_arrive_release();
        cluster_wait_acquire();
        if (active && warp < 4) {
            // Each row (maximum, sum, unnormalised O) goes straight from tensor memory into the shared
            // memory of the CTA that finishes it: remote stores stream, remote loads would each cost a
            // round trip.  Row r of the tile is finished by the CTA of chunk r / (128 / n_chunks).
            const int rows_per = kRowTile / plan.n_chunks;
            const int tid = warp * 32 + lane;
            const int row_in_tile = m64 ? (lane < 16 ? warp * 16 + lane : -1) : tid;
            const int rr = max(row_in_tile, 0);
            const int slot = chunk * rows_per + rr % rows_per;
            const uint32_t xo_remote = map_dsmem(smem_u32(k_smem), (uint32_t)(rr / rows_per));
            const uint32_t xs_remote = xo_remote + kRowTile * kD * 4;
            // rows beyond the tile's last query row and rows of unused nodes are not exchanged: the merge
            // writes zeros for the latter without reading anything
            const int push_row = rt * kRowTile + rr;
            const bool mine = rows_ready && row_in_tile >= 0 && push_row < plan.rows && push_row / G < n;
            tc_fence_after_sync();
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                uint32_t o[32];
                tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + cc * 32, o);
                tmem_ld_wait();
                if (mine) {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        st_dsmem_v4(xo_remote + (uint32_t)(slot * kD + (((cc * 8 + k) ^ (slot & 31)) << 2)) * 4,
                                    o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
                }
            }
            if (mine) {
                st_dsmem_f32(xs_remote + slot * 4, m_used);
                st_dsmem_f32(xs_remote + (kRowTile + slot) * 4, l);
            }
        }
        // all rows have landed where they are finished
        __syncwarp();
        cluster_arrive_release();
        cluster_wait_acquire();
        if (warp < 4) {
            const uint32_t xo_addr = smem_u32(k_smem);
            const MergeCtx mc{bt, plan, out, lse, xo_addr, xo_addr + kRowTile * kD * 4,
                              chunk, rt, b, kvh, n, tpc, tiles_total, warp, lane};
            if (plan.n_chunks == 2) merge_rows<2>(mc);
            else if (plan.n_chunks == 4) merge_rows<4>(mc);
            else merge_rows<8>(mc);
        }
    }
    if (!aligned) return;
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kTmaWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

static bool fill_layer(AttnLayer* ly, const sd_batch& bt, const sd_kv_layer& cache, const void* q,
                       const void* kt, const void* vt, void* out, float* lse) {
    const uint64_t cache_rows = (uint64_t)cache.num_blocks * bt.Hkv * kKeyTile;
    if (!encode_tmap_bf16_2d(&ly->k_cache, cache.k, cache_rows, kD, kD * 2, 64, kKeyTile, 128) ||
        !encode_tmap_bf16_2d(&ly->v_cache, cache.v, cache_rows, kD, kD * 2, 64, kKeyTile, 128))
        return false;
    const uint64_t dims[3] = {(uint64_t)kD, (uint64_t)bt.Hkv, (uint64_t)bt.B * bt.T_max};
    const uint64_t strides[2] = {(uint64_t)kD * 2, (uint64_t)bt.Hkv * kD * 2};
    const uint32_t box[3] = {64, 1, kKeyTile};
    if (!encode_tmap_bf16_3d(&ly->k_tree, kt, dims, strides, box, 128) ||
        !encode_tmap_bf16_3d(&ly->v_tree, vt, dims, strides, box, 128))
        return false;
    ly->q = static_cast<const uint16_t*>(q);
    ly->out = static_cast<__nv_bfloat16*>(out);
    ly->lse = lse;
    ly->num_blocks = cache.num_blocks;
    return true;
}

template <int NL>
sd_status launch_rows1(const AttnLayers<NL>& layers, const sd_batch& bt, float scale, const AttnPlan& plan,
                       int z_count, int32_t* dev_status, cudaStream_t st) {
    auto kern = attn_umma_kernel<NL>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttSmem) != cudaSuccess)
        return SD_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.n_chunks, plan.ctas_per_group, z_count);
    cfg.blockDim = dim3(kAttThreads);
    cfg.dynamicSmemBytes = kAttSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;      // the chunks of one row tile form a cluster
    attr[0].val.clusterDim.x = plan.n_chunks;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // The launch may begin while the kernel before it in the stream is still running (its CTAs take the
    // SM slots that one frees and do their set-up); the kernel waits for that kernel's completion before
    // it touches global memory.  Consecutive attention calls - one per layer - overlap their ends this way.
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, kern, layers, bt, scale * kLog2e, plan, dev_status) != cudaSuccess)
        return SD_ERR_CUDA;
    return SD_OK;
}
template sd_status launch_rows1<1>(const AttnLayers<1>&, const sd_batch&, float, const AttnPlan&, int, int32_t*,
                                   cudaStream_t);
template sd_status launch_rows1<kMaxLayersPerLaunch>(const AttnLayers<kMaxLayersPerLaunch>&, const sd_batch&, float,
                                                     const AttnPlan&, int, int32_t*, cudaStream_t);

// SM count of the current device (cached per device ordinal)
static int sm_count() {
    constexpr int kDevs = 64;
    static int cache[kDevs];
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return 148;
    if (dev < kDevs && cache[dev] > 0) return cache[dev];
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    if (dev < kDevs) cache[dev] = sms;
    return sms;
}

// The chunks of a row tile are merged inside a thread-block cluster, through shared memory:
// attention needs no global scratch (a nominal size keeps the argument checks uniform).
size_t attention_workspace_bytes(const sd_batch&) { return 256; }

// How many key chunks per sequence.
static AttnPlan make_plan(const sd_batch& bt, int n_layers, int sms) {
    AttnPlan p;
    const int G = bt.Hq / bt.Hkv;
    p.rows = bt.T_max * G;
    p.row_tiles = (p.rows + kRowTile - 1) / kRowTile;
    p.ctas_per_group = p.row_tiles;
    // Pick the chunk count that minimises (waves of CTAs) x (key tiles per CTA + fixed cost),
    // two CTAs being resident per SM.  Few waves are counted whole; many waves balance out.
    const int max_tiles = bt.max_blocks_per_seq;
    const int base = n_layers * bt.B * bt.Hkv * p.row_tiles;
    const int slots = 2 * sms;
    int n = 1;
    double best = 1e30;
    for (int c = 1; c <= kMaxChunks && c <= max_tiles; c *= 2) {   // 128 rows split evenly over the chunks
        const double w = (double)base * c / slots;
        double waves = (w <= 4.0) ? (double)((base * c + slots - 1) / slots) : w;
        // Without chunks, and for up to kSplitRounds whole rounds, the CTAs left over after the last whole
        // round go into a launch of their own, with chunks (launch_group): the partial round then costs
        // a fraction of a round.  (Longer launches run under the power cap, where this gained nothing.)
        if (c == 1 && w > 1.0 && base / slots < kSplitRounds) {
            const int rest = base % slots;
            int ct = 1;                                    // chunks of the remainder's launch
            while (2 * ct <= kMaxChunks && 2 * ct <= max_tiles && rest * 2 * ct <= slots) ct *= 2;
            waves = (double)(base / slots) + (rest == 0 ? 0.0 : (ct > 1 ? 1.0 / ct + 0.1 : 1.0));
        }
        // per CTA: its key tiles, a fixed cost of about three tiles, and the in-cluster merge: two to three
        // tiles' worth for clusters of two and four, about eleven for clusters of eight (measured: with
        // eight chunks a launch gains nothing over four unless it saves more than eight tiles per CTA)
        const int merge = (c == 1) ? 0 : (c == 2 ? 2 : (c == 4 ? 3 : 11));
        const double cost = waves * ((max_tiles + c - 1) / c + 3 + merge);
        if (cost < best - 1e-9) { best = cost; n = c; }
    }
    const TestKnobs knobs = test_knobs();
    if (knobs.chunks > 0 && knobs.chunks <= max_tiles) n = knobs.chunks;     // test hook
    p.n_chunks = n;
    p.n_layers = n_layers;
    p.ranked = (bt.B > 1 && bt.B <= 64 && (long long)base * n > slots) ? 1 : 0;
    p.z0 = 0;
    p.wait_cycles = knobs.wait_cycles;
    p.withhold = knobs.withhold;
    return p;
}

template <int NL>
static sd_status launch_group(const AttnLayers<NL>& layers, int n_layers, const sd_batch& bt, float scale,
                              int32_t* dev_status, cudaStream_t st) {
    AttnPlan plan = make_plan(bt, n_layers, sm_count());
    const int Z = n_layers * bt.B * bt.Hkv;
    // A launch of whole-sequence CTAs that runs for more than one round ends on a partial round, in which
    // the CTAs left over would each work through a whole sequence while most of the GPU idles.  They go
    // into a second launch of the same kernel with the keys split into chunks (a cluster per row tile),
    // so that the remainder also spreads over the SMs and takes a fraction of a round.  (In a ranked
    // launch these are the shortest sequences.)
    const int slots = 2 * sm_count();
    const long long ctas = (long long)Z * plan.row_tiles;
    if (plan.n_chunks == 1 && ctas > slots && ctas / slots < kSplitRounds && test_knobs().chunks == 0) {
        const int z_main = (int)((ctas / slots) * slots / plan.row_tiles);
        const int z_rest = Z - z_main;
        int c = 1;
        while (2 * c <= kMaxChunks && 2 * c <= bt.max_blocks_per_seq &&
               (long long)z_rest * plan.row_tiles * 2 * c <= slots) c *= 2;
        if (z_main > 0 && z_rest > 0 && c > 1) {
            const sd_status s = launch_rows1<NL>(layers, bt, scale, plan, z_main, dev_status, st);
            if (s != SD_OK) return s;
            plan.z0 = z_main;
            plan.n_chunks = c;
            return launch_rows1<NL>(layers, bt, scale, plan, z_rest, dev_status, st);
        }
    }
    return launch_rows1<NL>(layers, bt, scale, plan, Z, dev_status, st);
}

// One launch per group of layers: at most kMaxLayersPerLaunch descriptors fit the kernel's
// parameter space and gridDim.z is limited to 65535.
sd_status launch_attention_layers(const sd_batch& bt, const sd_kv_layer* caches, int L,
                                  const void* const* q, const void* const* kt, const void* const* vt,
                                  float scale, void* const* out, float* const* lse,
                                  int32_t* dev_status, cudaStream_t st) {
    const int per_layer_z = bt.B * bt.Hkv;
    if (per_layer_z > 65535) return SD_ERR_UNSUPPORTED;
    int group = 65535 / per_layer_z;
    if (group > kMaxLayersPerLaunch) group = kMaxLayersPerLaunch;
    for (int l0 = 0; l0 < L; l0 += group) {
        const int nl = (L - l0 < group) ? (L - l0) : group;
        if (nl == 1) {
            AttnLayers<1> one;
            if (!fill_layer(&one.l[0], bt, caches[l0], q[l0], kt[l0], vt[l0], out[l0], lse ? lse[l0] : nullptr))
                return SD_ERR_CUDA;
            sd_status s = launch_group<1>(one, 1, bt, scale, dev_status, st);
            if (s != SD_OK) return s;
        } else {
            AttnLayers<kMaxLayersPerLaunch> many;
            for (int i = 0; i < nl; ++i)
                if (!fill_layer(&many.l[i], bt, caches[l0 + i], q[l0 + i], kt[l0 + i], vt[l0 + i], out[l0 + i],
                                lse ? lse[l0 + i] : nullptr))
                    return SD_ERR_CUDA;
            for (int i = nl; i < kMaxLayersPerLaunch; ++i) many.l[i] = many.l[0];
            sd_status s = launch_group<kMaxLayersPerLaunch>(many, nl, bt, scale, dev_status, st);
            if (s != SD_OK) return s;
        }
    }
    return SD_OK;
}

sd_status launch_attention(const sd_batch& bt, const sd_kv_layer& cache, const void* q,
                           const void* kt, const void* vt, float scale, void* out, float* lse,
                           void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t st) {
    (void)ws;
    if (ws_bytes < attention_workspace_bytes(bt)) return SD_ERR_WORKSPACE;
    return launch_attention_layers(bt, &cache, 1, &q, &kt, &vt, scale, &out, &lse, dev_status, st);
}

}  // namespace sdv
