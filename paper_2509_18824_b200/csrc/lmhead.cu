// LM-head projection with fused arg-max on the 5th-generation tensor cores.
//
// logits^T = W . hidden^T is computed tile by tile with the vocabulary along
// the MMA M dimension (TMEM lanes) and the hidden rows along N (TMEM columns):
// every CTA streams its own slab of W exactly once (TMA, 128-byte swizzle)
// while the small hidden matrix is re-read from L2.  The accumulator never
// leaves TMEM: the epilogue warps reduce each column over the 128 vocabulary
// lanes (max + lowest index) and keep a running best per hidden row; only
// (max, index) pairs per CTA reach memory, and a tiny kernel merges them.
#include <atomic>
#include "tree_device.cuh"
#include "sm100.cuh"

namespace sdv {
using namespace sm100;

constexpr int kBM = 128;            // vocabulary rows per tile (MMA M)
constexpr int kEpiWarps = 8;        // two epilogue warps per TMEM lane quadrant: even and odd 32-column chunks
constexpr int kTmaWarpLm = kEpiWarps, kMmaWarpLm = kEpiWarps + 1;
constexpr int kLmThreads = kEpiWarps * 32 + 32 + 1;   // epilogue warps, TMA producer warp, ONE thread: MMA issuer
                                    // (a one-thread warp keeps the issue loop in uniform control flow, so
                                    //  the MMA descriptors stay in uniform registers)
constexpr int kMaxCols = kLmMaxCols; // hidden rows per launch (TMEM columns)
constexpr int kMaxCtas = 256;
constexpr int kMaxStages = 8;
constexpr int kSmemBudget = 227 * 1024 - 2048;

struct LmParams {
    int rows;          // hidden rows handled by this launch (<= 512)
    int row0;          // index of the first one
    int Hd, V;
    int n_parts;       // MMA instructions along N per k-step (1 or 2)
    int part_n;        // N of each (multiple of 16, <= 256)
    int n_pad;         // n_parts * part_n
    int buf_stride;    // TMEM columns per accumulator buffer
    int acc_bufs;      // 1 or 2 accumulator buffers
    int tmem_cols;     // allocation (power of two >= 32)
    int n_tiles;       // vocabulary tiles
    int stages;
    int32_t* part_key; // [gridDim.x][kMaxCols] order-preserving integer image of the max logit
    int32_t* part_idx; // [gridDim.x][kMaxCols]
    // soft-max statistics (sampling at a temperature): c2 = log2(e) / temperature, 0 = not wanted
    float c2;
    float* part_ref;   // [gridDim.x][kMaxCols] reference logit of the partial sum
    float* part_sum;   // [gridDim.x][kMaxCols] sum over the CTA's vocabulary rows of 2^((logit - ref) * c2)
    // probability output (residual draw of the sampled acceptance): when mass_out is set, the epilogue
    // stores exp(logit * inv_temp - col_lse[row]) for every (row, vocabulary entry) instead of reducing
    // per 32 vocabulary rows and hidden row: (group maximum, sum of 2^((logit - maximum) * c2)), optional;
    // the residual draw of the sampled acceptance finds its token from these without a second pass over W
    float2* group_stats;    // [ceil(V / 32)][M_total]
    int M_total;
    float* mass_out;        // [rows of the call][V]
    float* logit_out;       // statistics pass only, optional: the raw logits, [M_total][V] (small M: chain decoding)
    const float* col_lse;   // [rows of the call]
    float inv_temp;
    long long wait_cycles;  // bound of every barrier wait, in SM cycles
    int withhold;           // test hook (single-CTA kernel): the first tile's "accumulator complete" is never signalled
};

size_t lmhead_workspace_bytes(int M, int V) {
    (void)M; (void)V;
    return (size_t)kMaxCtas * kMaxCols * 2 * sizeof(int32_t);
}
// the fused tail also parks the acceptance outputs of its non-writing CTAs: per layer
// 2 * B + 2 * B * T_max <= 4 * 512 words, for up to 64 layers
size_t tail_workspace_bytes(int M, int V) {
    return lmhead_workspace_bytes(M, V) + (size_t)kLayersPerLaunch * 4 * kMaxCols * sizeof(int32_t);
}
// soft-max statistics: two more per-CTA tables (reference, partial sum), behind the tail's area
size_t stats_workspace_bytes(int M, int V) {
    return tail_workspace_bytes(M, V) + (size_t)kMaxCtas * kMaxCols * 2 * sizeof(float);
}

// float -> int whose signed order equals the float order (-0 folded onto +0)
__device__ __forceinline__ int32_t ordered_key(uint32_t bits) {
    int32_t b = (int32_t)bits;
    b = (b < 0) ? (b ^ 0x7fffffff) : b;
    return (b == -1) ? 0 : b;            // -0.0f maps to -1 above; fold it onto +0.0f
}

__device__ __forceinline__ float redux_max_f32(float v) {
    float d;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(d) : "f"(v));
    return d;
}

// element `lane` of a 32-entry register array, by a binary tree of selects on the lane's bits
// (register arrays cannot be indexed by a run-time value)
template <typename T>
__device__ __forceinline__ T pick_lane(const T (&x)[32], int lane) {
    T a[16], b[8], c[4], d[2];
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = (lane & 16) ? x[i + 16] : x[i];
#pragma unroll
    for (int i = 0; i < 8; ++i) b[i] = (lane & 8) ? a[i + 8] : a[i];
#pragma unroll
    for (int i = 0; i < 4; ++i) c[i] = (lane & 4) ? b[i + 4] : b[i];
#pragma unroll
    for (int i = 0; i < 2; ++i) d[i] = (lane & 2) ? c[i + 2] : c[i];
    return (lane & 1) ? d[1] : d[0];
}

// Arg-max over the 32 lanes (vocabulary rows) of each of 32 accumulator columns (hidden rows):
// lane j ends up with column j's maximum and the lowest vocabulary row attaining it.  The passes
// are kept apart on purpose: 32 independent warp reductions are in flight together, then 32
// independent votes; interleaved per column, every reduction's latency (and then every vote's)
// would be paid one after the other.
__device__ __forceinline__ void column_argmax32(const uint32_t (&r)[32], bool v_ok, int v_base, int lane,
                                                float& cv, int32_t& ci) {
    float v[32], mx[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = v_ok ? __uint_as_float(r[j]) : -INFINITY;
#pragma unroll
    for (int j = 0; j < 32; ++j) mx[j] = redux_max_f32(v[j]);
    uint32_t who[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) who[j] = __ballot_sync(0xffffffffu, v[j] == mx[j]);
    cv = pick_lane(mx, lane);
    ci = v_base + (__ffs(pick_lane(who, lane)) - 1);
}

// Sum over the 32 lanes of each of 32 per-lane values: lane j receives sum_lanes x[j].  Five
// exchange steps; in each a lane keeps the half of its values whose column index has the step's
// bit equal to its own lane bit and hands the other half to its partner (fixed order of additions).
__device__ __forceinline__ float transpose_sum32(const float (&x)[32], int lane) {
    float a[16], b[8], c[4], d[2];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float keep = (lane & 16) ? x[i + 16] : x[i], send = (lane & 16) ? x[i] : x[i + 16];
        a[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float keep = (lane & 8) ? a[i + 8] : a[i], send = (lane & 8) ? a[i] : a[i + 8];
        b[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float keep = (lane & 4) ? b[i + 4] : b[i], send = (lane & 4) ? b[i] : b[i + 4];
        c[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const float keep = (lane & 2) ? c[i + 2] : c[i], send = (lane & 2) ? c[i] : c[i + 2];
        d[i] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
    }
    const float keep = (lane & 1) ? d[1] : d[0], send = (lane & 1) ? d[0] : d[1];
    return keep + __shfl_xor_sync(0xffffffffu, send, 1);
}

// The same arg-max plus, per column, sum over the 32 vocabulary rows of 2^((logit - column max) * c2):
// lane j receives column j's sum in cs.
__device__ __forceinline__ void column_argmax_stats32(const uint32_t (&r)[32], bool v_ok, int v_base, int lane,
                                                      float c2, float& cv, int32_t& ci, float& cs) {
    float v[32], mx[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = v_ok ? __uint_as_float(r[j]) : -INFINITY;
#pragma unroll
    for (int j = 0; j < 32; ++j) mx[j] = redux_max_f32(v[j]);
    uint32_t who[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) who[j] = __ballot_sync(0xffffffffu, v[j] == mx[j]);
    cv = pick_lane(mx, lane);
    ci = v_base + (__ffs(pick_lane(who, lane)) - 1);
    float e[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) e[j] = (v[j] == -INFINITY) ? 0.f : ex2_lm((v[j] - mx[j]) * c2);
    cs = transpose_sum32(e, lane);
}

// ---------------------------------------------------------------------------
// Epilogue shared by the one-CTA and the two-CTA kernel.  Warp w of the eight epilogue warps works on
// TMEM lanes 32 * (w & 3) .. +31 (the only ones it may read) and on the 32-column chunks of parity
// w >> 2; per (warp, column) it keeps a running best (value, vocabulary row) and, for the soft-max
// statistics, a running (reference, sum).
// ---------------------------------------------------------------------------
struct EpiState {
    float best_val[kMaxCols / 64];
    int32_t best_idx[kMaxCols / 64];
    float run_ref[kMaxCols / 64], run_sum[kMaxCols / 64];
};

__device__ __forceinline__ void epi_init(EpiState& e) {
#pragma unroll
    for (int c = 0; c < kMaxCols / 64; ++c) {
        e.best_val[c] = -INFINITY; e.best_idx[c] = 0x7fffffff; e.run_ref[c] = -INFINITY; e.run_sum[c] = 0.f;
    }
}

// one accumulator tile (128 vocabulary rows from v_base - 32 * quad on; this warp's 32 of them start at v_base)
__device__ __forceinline__ void epi_tile(const LmParams& p, EpiState& e, uint32_t taddr, int v_base, int lane, int par) {
    const bool stats = p.c2 > 0.f;
    const bool v_ok = (v_base + lane) < p.V;
#pragma unroll
    for (int h = 0; h < kMaxCols / 64; ++h) {
        const int c = 2 * h + par;                 // this warp's chunk of the pair (2h, 2h + 1)
        if (c * 32 < p.n_pad) {
            uint32_t r[32];
            tmem_ld32(taddr + c * 32, r);
            tmem_ld_wait();
            float cv;
            int32_t ci;
            if (p.mass_out) {
                if (v_ok) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int row = c * 32 + j;
                        if (row < p.rows)
                            p.mass_out[(size_t)(p.row0 + row) * p.V + v_base + lane] =
                                __expf(__uint_as_float(r[j]) * p.inv_temp - __ldg(p.col_lse + p.row0 + row));
                    }
                }
                continue;
            }
            if (stats) {
                if (p.logit_out && v_ok) {             // the raw logits, one running address (few rows: chain decoding)
                    float* dst = p.logit_out + (size_t)(p.row0 + c * 32) * p.V + v_base + lane;
                    const int lim = p.rows - c * 32;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (j < lim) *dst = __uint_as_float(r[j]);
                        dst += p.V;
                    }
                }
                float cs;
                column_argmax_stats32(r, v_ok, v_base, lane, p.c2, cv, ci, cs);
                merge_sumexp(e.run_ref[h], e.run_sum[h], cv, cs, p.c2);
                if (p.group_stats && v_base < p.V && c * 32 + lane < p.rows)
                    p.group_stats[(size_t)(v_base >> 5) * p.M_total + p.row0 + c * 32 + lane] = make_float2(cv, cs);

            } else {
                column_argmax32(r, v_ok, v_base, lane, cv, ci);
            }
            if (cv > e.best_val[h]) { e.best_val[h] = cv; e.best_idx[h] = ci; }
        }
    }
}

// After the last tile: the four lane quadrants' results are merged through shared memory (the pipeline
// stages are idle by now: the last accumulator was complete, so every copy has landed and every MMA has
// read it) and this CTA's row of the candidate tables is written.
__device__ __forceinline__ void epi_finish(const LmParams& p, const EpiState& e, uint8_t* smem, int quad, int par,
                                           int lane, bool ok, int32_t* status) {
    const bool stats = p.c2 > 0.f;
    asm volatile("bar.sync 1, %0;" ::"n"(kEpiWarps * 32) : "memory");
    int32_t* red_key = reinterpret_cast<int32_t*>(smem);
    int32_t* red_idx = red_key + 4 * kMaxCols;
    float* red_ref = reinterpret_cast<float*>(red_idx + 4 * kMaxCols);
    float* red_sum = red_ref + 4 * kMaxCols;
#pragma unroll
    for (int h = 0; h < kMaxCols / 64; ++h) {
        red_key[quad * kMaxCols + (2 * h + par) * 32 + lane] = ordered_key(__float_as_uint(e.best_val[h]));
        red_idx[quad * kMaxCols + (2 * h + par) * 32 + lane] = e.best_idx[h];
        if (stats) {
            red_ref[quad * kMaxCols + (2 * h + par) * 32 + lane] = e.run_ref[h];
            red_sum[quad * kMaxCols + (2 * h + par) * 32 + lane] = e.run_sum[h];
        }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kEpiWarps * 32) : "memory");
    for (int col = threadIdx.x; col < kMaxCols; col += kEpiWarps * 32) {
        int32_t k = red_key[col], i = red_idx[col];
#pragma unroll
        for (int w = 1; w < 4; ++w) {
            const int32_t k2 = red_key[w * kMaxCols + col], i2 = red_idx[w * kMaxCols + col];
            if (k2 > k || (k2 == k && i2 < i)) { k = k2; i = i2; }
        }
        if (!ok && col == (int)threadIdx.x) set_status(status, SD_ERR_TIMEOUT);
        p.part_key[(size_t)blockIdx.x * kMaxCols + col] = ok ? k : INT32_MIN;
        p.part_idx[(size_t)blockIdx.x * kMaxCols + col] = i;
        if (stats) {
            float rf = red_ref[col], sm = red_sum[col];
#pragma unroll
            for (int w = 1; w < 4; ++w) merge_sumexp(rf, sm, red_ref[w * kMaxCols + col], red_sum[w * kMaxCols + col], p.c2);
            p.part_ref[(size_t)blockIdx.x * kMaxCols + col] = rf;
            p.part_sum[(size_t)blockIdx.x * kMaxCols + col] = sm;
        }
    }
}

template <int BK>
__global__ void __launch_bounds__(kLmThreads, 1)
lmhead_umma_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmH,
                   const LmParams p, int32_t* status) {
    constexpr int kSwz = BK * 2;                 // bytes per smem row = swizzle span
    constexpr int kGroup = 8 * kSwz;             // 8-row swizzle group
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int a_bytes = kBM * kSwz;
    const int stage_bytes = a_bytes + p.n_pad * kSwz;

    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t tmem_full[2];
    __shared__ __align__(8) uint64_t tmem_empty[2];
    __shared__ __align__(8) uint64_t mma_idle;               // unwinding only: every MMA issued so far has completed
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform for the compiler
    const int lane = threadIdx.x & 31;
    const int kblocks = p.Hd / BK;
    const int my_tiles = (p.n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full[b], 1); mbar_init(&tmem_empty[b], kEpiWarps); }
        mbar_init(&mma_idle, 1);
        fence_barrier_init();
    }
    if (warp == kTmaWarpLm) {          // a full warp
        tmem_alloc(&tmem_base_slot, (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    if (warp == kTmaWarpLm && lane == 0) { prefetch_tensormap(&tmW); prefetch_tensormap(&tmH); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == kTmaWarpLm) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first();
            const uint64_t pol_h = policy_evict_last();
            int it = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int v0 = ((int)blockIdx.x + t * (int)gridDim.x) * kBM;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
                    if (!mbar_wait(&empty_bar[s], ph ^ 1u, &abort_flag, p.wait_cycles)) { ok = false; break; }
                    uint8_t* a = smem + (size_t)s * stage_bytes;
                    mbar_arrive_expect_tx(&full_bar[s], (uint32_t)stage_bytes);
                    tma_load_2d(a, &tmW, kb * BK, v0, &full_bar[s], pol_w);
                    for (int part = 0; part < p.n_parts; ++part)
                        tma_load_2d(a + a_bytes + (size_t)part * p.part_n * kSwz, &tmH, kb * BK,
                                    p.row0 + part * p.part_n, &full_bar[s], pol_h);
                }
            }
            if (!ok) {
                set_status(status, SD_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let copies in flight land
            }
        }
    } else if (warp == kMmaWarpLm) {
        // ------------------------------------------------ MMA issuer (this warp is one thread)
        {
            const uint32_t idesc = make_idesc_bf16(kBM, p.part_n, false, false);
            int it = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int buf = t % p.acc_bufs;
                const uint32_t use = (uint32_t)(t / p.acc_bufs);
                if (!mbar_wait(&tmem_empty[buf], (use & 1u) ^ 1u, &abort_flag, p.wait_cycles)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d0 = tmem_base + (uint32_t)(buf * p.buf_stride);
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
                    if (!mbar_wait(&full_bar[s], ph, &abort_flag, p.wait_cycles)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint32_t b_addr = a_addr + (uint32_t)a_bytes;
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        const uint64_t adesc = make_smem_desc(a_addr + k * 32, 16, kGroup, kSwz);
                        for (int part = 0; part < p.n_parts; ++part) {
                            const uint64_t bdesc =
                                make_smem_desc(b_addr + (uint32_t)(part * p.part_n * kSwz) + k * 32, 16, kGroup, kSwz);
                            mma_ss(d0 + (uint32_t)(part * p.part_n), adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
                        }
                    }
                    mma_commit(&empty_bar[s]);            // stage reusable once these MMAs have read it
                }
                if (ok && !(p.withhold && t == 0)) mma_commit(&tmem_full[buf]);       // accumulator complete
            }
            if (!ok || p.withhold) {
                // unwinding: nothing may give tensor memory back while an MMA issued above still runs
                if (!ok) set_status(status, SD_ERR_TIMEOUT);
                mma_commit(&mma_idle);
                mbar_wait_plain(&mma_idle, 0, p.wait_cycles);
            }
        }
    } else {
        // ------------------------------------------------ epilogue warps 0..7
        const int quad = warp & 3, par = warp >> 2;
        EpiState e;
        epi_init(e);
        bool ok = true;
        for (int t = 0; t < my_tiles && ok; ++t) {
            const int buf = t % p.acc_bufs;
            const uint32_t use = (uint32_t)(t / p.acc_bufs);
            if (!mbar_wait(&tmem_full[buf], use & 1u, &abort_flag, p.wait_cycles)) { ok = false; break; }
            tc_fence_after_sync();
            const int v_base = ((int)blockIdx.x + t * (int)gridDim.x) * kBM + quad * 32;
            epi_tile(p, e, tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * p.buf_stride), v_base, lane, par);
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tmem_empty[buf]);
        }
        epi_finish(p, e, smem, quad, par, lane, ok, status);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kTmaWarpLm) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// ---------------------------------------------------------------------------
// Two-CTA version (cta_group::2): a cluster of two CTAs works on 256 vocabulary
// rows at a time.  Each CTA streams its own 128 rows of W and HALF of the hidden
// rows of every k-step; one tcgen05.mma issued by the leader CTA multiplies both
// halves against both W slabs and fills the accumulators in both CTAs' TMEM.
// The hidden matrix is therefore re-read from L2 half as often per W byte.
// ---------------------------------------------------------------------------
template <int BK, int NPARTS>
__global__ void __launch_bounds__(kLmThreads, 1)
lmhead_umma_pair_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmH,
                        const LmParams p, int32_t* status) {
    constexpr int kSwz = BK * 2;
    constexpr int kGroup = 8 * kSwz;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int a_bytes = kBM * kSwz;
    const int half_n = p.part_n / 2;                          // hidden rows of one MMA held by this CTA
    const int stage_bytes = a_bytes + p.n_parts * half_n * kSwz;

    __shared__ __align__(8) uint64_t full_bar[kMaxStages];   // used in the leader: both CTAs' loads
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];  // in each CTA: stage consumed
    __shared__ __align__(8) uint64_t tmem_full[2];           // in each CTA: accumulator complete
    __shared__ __align__(8) uint64_t tmem_empty[2];          // used in the leader: 8 epilogue warps done
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform for the compiler
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                  // 0 = leader
    const int pair = blockIdx.x >> 1;
    const int n_pairs = gridDim.x >> 1;
    const int kblocks = p.Hd / BK;
    const int my_tiles = (p.n_tiles - pair + n_pairs - 1) / n_pairs;   // tiles of 256 vocabulary rows

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full[b], 1); mbar_init(&tmem_empty[b], 2 * kEpiWarps); }
        fence_barrier_init();
    }
    if (warp == kTmaWarpLm) {          // a full warp
        tmem_alloc_pair(&tmem_base_slot, (uint32_t)p.tmem_cols);
        tmem_relinquish_pair();
    }
    if (warp == kTmaWarpLm && lane == 0) { prefetch_tensormap(&tmW); prefetch_tensormap(&tmH); }
    tc_fence_before_sync();
    __syncthreads();
    cluster_arrive_release();          // the partner's barriers exist before anything signals them
    cluster_wait_acquire();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == kTmaWarpLm) {
        // ------------------------------------------------ TMA producer (one per CTA)
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first();
            const uint64_t pol_h = policy_evict_last();
            int it = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int v0 = ((pair + t * n_pairs) * 2 + (int)rank) * kBM;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
                    if (!mbar_wait(&empty_bar[s], ph ^ 1u, &abort_flag, p.wait_cycles)) { ok = false; break; }
                    uint8_t* a = smem + (size_t)s * stage_bytes;
                    if (rank == 0) mbar_arrive_expect_tx(&full_bar[s], 2u * (uint32_t)stage_bytes);
                    const uint32_t bar = map_dsmem(smem_u32(&full_bar[s]), 0);     // the leader's barrier
                    tma_load_2d_pair(a, &tmW, kb * BK, v0, bar, pol_w);
                    for (int part = 0; part < p.n_parts; ++part)
                        tma_load_2d_pair(a + a_bytes + (size_t)part * half_n * kSwz, &tmH, kb * BK,
                                         p.row0 + part * p.part_n + (int)rank * half_n, bar, pol_h);
                }
            }
            if (!ok) {
                set_status(status, SD_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let copies in flight land
            }
        }
    } else if (warp == kMmaWarpLm) {
        // ------------------------------------------------ MMA issuer (leader CTA only; this warp is one thread)
        if (rank == 0) {
            const uint32_t idesc = make_idesc_bf16(2 * kBM, p.part_n, false, false);
            const uint32_t part_step = (uint32_t)(half_n * kSwz) >> 4;   // next part's B rows, in descriptor units
            int it = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int buf = t % p.acc_bufs;
                const uint32_t use = (uint32_t)(t / p.acc_bufs);
                if (!mbar_wait(&tmem_empty[buf], (use & 1u) ^ 1u, &abort_flag, p.wait_cycles)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d0 = tmem_base + (uint32_t)(buf * p.buf_stride);
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
                    if (!mbar_wait(&full_bar[s], ph, &abort_flag, p.wait_cycles)) { ok = false; break; }
                    tc_fence_after_sync();
                    // descriptors of the stage; k-steps and parts only move the 16-byte-granular start address
                    const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint64_t adesc0 = make_smem_desc(a_addr, 16, kGroup, kSwz);
                    const uint64_t bdesc0 = make_smem_desc(a_addr + (uint32_t)a_bytes, 16, kGroup, kSwz);
                    const uint32_t first = (kb != 0) ? 1u : 0u;
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
#pragma unroll
                        for (int part = 0; part < NPARTS; ++part) {
                            mma_ss_pair(d0 + (uint32_t)(part * p.part_n), adesc0 + (uint64_t)(k * 2),
                                        bdesc0 + (uint64_t)(part * part_step + k * 2), idesc, k != 0 ? 1u : first);
                        }
                    }
                    mma_commit_pair(&empty_bar[s], 3);        // both CTAs may refill this stage
                }
                if (ok) mma_commit_pair(&tmem_full[buf], 3);  // accumulators complete in both CTAs
            }
            if (!ok) set_status(status, SD_ERR_TIMEOUT);
        }
    } else {
        // ------------------------------------------------ epilogue warps 0..7
        const int quad = warp & 3, par = warp >> 2;
        EpiState e;
        epi_init(e);
        bool ok = true;
        for (int t = 0; t < my_tiles && ok; ++t) {
            const int buf = t % p.acc_bufs;
            const uint32_t use = (uint32_t)(t / p.acc_bufs);
            if (!mbar_wait(&tmem_full[buf], use & 1u, &abort_flag, p.wait_cycles)) { ok = false; break; }
            tc_fence_after_sync();
            const int v_base = ((pair + t * n_pairs) * 2 + (int)rank) * kBM + quad * 32;
            epi_tile(p, e, tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * p.buf_stride), v_base, lane, par);
            tc_fence_before_sync();
            __syncwarp();
            // (the accumulator reads above have completed: tcgen05.wait::ld; a CTA-scope release is enough,
            //  and a cluster-scope one costs on the order of a thousand cycles per arrival)
            if (lane == 0) mbar_arrive_remote_light(map_dsmem(smem_u32(&tmem_empty[buf]), 0));
        }
        epi_finish(p, e, smem, quad, par, lane, ok, status);
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_arrive_release();          // neither CTA leaves while the other may still signal it
    cluster_wait_acquire();
    if (warp == kTmaWarpLm) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// one thread per hidden row: merge the per-CTA candidates (lowest index on ties)
__global__ void lmhead_merge_kernel(const int32_t* __restrict__ part_key, const int32_t* __restrict__ part_idx,
                                    int n_ctas, int rows, int row0, int32_t* __restrict__ argmax,
                                    float* __restrict__ maxlogit) {
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    if (col >= rows) return;
    int32_t k = INT32_MIN, i = 0x7fffffff;
    for (int c = 0; c < n_ctas; ++c) {
        const int32_t k2 = part_key[(size_t)c * kMaxCols + col], i2 = part_idx[(size_t)c * kMaxCols + col];
        if (k2 > k || (k2 == k && i2 < i)) { k = k2; i = i2; }
    }
    argmax[row0 + col] = i;
    if (maxlogit) maxlogit[row0 + col] = key_to_float(k);
}

// the same merge plus log sum exp(logit / temperature) of every hidden row (natural log);
// eight threads per row share the CTAs' partials and combine through shuffles (fixed order)
__global__ void __launch_bounds__(256)
lmhead_merge_stats_kernel(const int32_t* __restrict__ part_key, const int32_t* __restrict__ part_idx,
                          const float* __restrict__ part_ref, const float* __restrict__ part_sum,
                          int n_ctas, int rows, int row0, float c2, int32_t* __restrict__ argmax,
                          float* __restrict__ maxlogit, float* __restrict__ lse) {
    const int col = blockIdx.x * 32 + (threadIdx.x >> 3), sub = threadIdx.x & 7;
    int32_t k, i;
    const float row_lse = merge_row_stats(part_key, part_idx, part_ref, part_sum, n_ctas, kMaxCols, col, col < rows, sub, c2, k, i);
    if (col < rows && sub == 0) {
        if (argmax) argmax[row0 + col] = i;
        if (maxlogit) maxlogit[row0 + col] = key_to_float(k);
        lse[row0 + col] = row_lse;
    }
}

static int round_up(int x, int m) { return (x + m - 1) / m * m; }

// tiles_only_ctas != nullptr (M <= 512 required): launch only the tile kernel and report how many
// CTAs filled the candidate tables; the caller merges them itself (the fused tail kernel).
static sd_status launch_lmhead_impl(const void* hidden, const void* W, int M, int Hd, int V,
                                    int32_t* argmax, float* maxlogit, void* ws, size_t ws_bytes,
                                    int32_t* dev_status, cudaStream_t st, int* tiles_only_ctas,
                                    float inv_temp = 0.f, float* lse = nullptr,
                                    float* mass_out = nullptr, const float* col_lse = nullptr,
                                    float* group_stats = nullptr, float* logit_out = nullptr) {
    if (ws_bytes < (lse ? stats_workspace_bytes(M, V) : lmhead_workspace_bytes(M, V))) return SD_ERR_WORKSPACE;
    if (tiles_only_ctas && M > kMaxCols) return SD_ERR_UNSUPPORTED;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return SD_ERR_CUDA;

    const int n_blocks = (M + kMaxCols - 1) / kMaxCols;
    const int rows_per_block = round_up((M + n_blocks - 1) / n_blocks, 16);
    for (int rb = 0; rb < n_blocks; ++rb) {
        LmParams p;
        p.row0 = rb * rows_per_block;
        p.rows = (M - p.row0 < rows_per_block) ? (M - p.row0) : rows_per_block;
        p.Hd = Hd; p.V = V;
        const int n16 = round_up(p.rows, 16);
        p.n_parts = (n16 > 256) ? 2 : 1;
        p.part_n = round_up((n16 + p.n_parts - 1) / p.n_parts, 16);
        p.n_pad = p.n_parts * p.part_n;
        p.buf_stride = round_up(p.n_pad, 32);
        p.acc_bufs = (2 * p.buf_stride <= kMaxCols) ? 2 : 1;
        int cols = 32;
        while (cols < p.acc_bufs * p.buf_stride) cols *= 2;
        p.tmem_cols = cols;
        p.n_tiles = (V + kBM - 1) / kBM;
        // Two-CTA tiles whenever a pair has work (the common case); rows per MMA part must then
        // split evenly over the two CTAs in whole 8-row swizzle groups.
        const bool pair = (sms >= 2) && (V > kBM);
        if (pair) {
            p.part_n = round_up(p.part_n, 16);
            p.n_tiles = (V + 2 * kBM - 1) / (2 * kBM);
        }
        const int b_rows = pair ? p.n_pad / 2 : p.n_pad;      // hidden rows staged per CTA and k-step
        // contraction step: 64 (128-byte swizzle) while at least four stages fit, else 32
        const int stage64 = (kBM + b_rows) * 128;
        const int bk = (4 * stage64 <= kSmemBudget) ? 64 : 32;
        const int stage_bytes = (kBM + b_rows) * bk * 2;
        int stages = kSmemBudget / stage_bytes;
        if (stages > kMaxStages) stages = kMaxStages;
        if (stages < 2) return SD_ERR_UNSUPPORTED;
        p.stages = stages;
        p.part_key = static_cast<int32_t*>(ws);
        p.part_idx = p.part_key + (size_t)kMaxCtas * kMaxCols;
        p.c2 = lse ? inv_temp * 1.4426950408889634f : 0.f;
        p.part_ref = reinterpret_cast<float*>(static_cast<char*>(ws) + tail_workspace_bytes(M, V));
        p.part_sum = p.part_ref + (size_t)kMaxCtas * kMaxCols;
        p.mass_out = mass_out; p.col_lse = col_lse; p.inv_temp = inv_temp;
        const TestKnobs knobs = test_knobs();
        p.wait_cycles = knobs.wait_cycles;
        p.withhold = knobs.withhold;
        p.group_stats = reinterpret_cast<float2*>(group_stats); p.M_total = M;
        p.logit_out = logit_out;

        CUtensorMap tmW, tmH;
        if (!encode_tmap_bf16_2d(&tmW, W, (uint64_t)V, (uint64_t)Hd, (uint64_t)Hd * 2, (uint32_t)bk, kBM, bk * 2))
            return SD_ERR_CUDA;
        if (!encode_tmap_bf16_2d(&tmH, hidden, (uint64_t)M, (uint64_t)Hd, (uint64_t)Hd * 2, (uint32_t)bk,
                                 (uint32_t)(pair ? p.part_n / 2 : p.part_n), bk * 2))
            return SD_ERR_CUDA;
        int grid = sms < kMaxCtas ? sms : kMaxCtas;
        const size_t dyn = (size_t)stages * stage_bytes + 1024;
        if (pair) {
            grid &= ~1;
            if (grid > 2 * p.n_tiles) grid = 2 * p.n_tiles;
            if (p.n_pad > 128) {
                // Tensor-bound sizes: the slowest pair sets the time (ceil(tiles / pairs) rounds), so use
                // the fewest pairs that still finish in that many rounds; the SMs left idle cost no time
                // and leave their share of the power budget to the others.
                const int rounds = (p.n_tiles + grid / 2 - 1) / (grid / 2);
                grid = 2 * ((p.n_tiles + rounds - 1) / rounds);
            }
            auto kern = (bk == 64) ? (p.n_parts == 2 ? lmhead_umma_pair_kernel<64, 2> : lmhead_umma_pair_kernel<64, 1>)
                                   : (p.n_parts == 2 ? lmhead_umma_pair_kernel<32, 2> : lmhead_umma_pair_kernel<32, 1>);
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
                return SD_ERR_CUDA;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(grid);
            cfg.blockDim = dim3(kLmThreads);
            cfg.dynamicSmemBytes = dyn;
            cfg.stream = st;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 2;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            if (cudaLaunchKernelEx(&cfg, kern, tmW, tmH, p, dev_status) != cudaSuccess) return SD_ERR_CUDA;
        } else {
            if (grid > p.n_tiles) grid = p.n_tiles;
            auto kern = (bk == 64) ? lmhead_umma_kernel<64> : lmhead_umma_kernel<32>;
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
                return SD_ERR_CUDA;
            kern<<<grid, kLmThreads, dyn, st>>>(tmW, tmH, p, dev_status);
            if (cudaGetLastError() != cudaSuccess) return SD_ERR_CUDA;
        }
        if (tiles_only_ctas) {
            *tiles_only_ctas = grid;
            return SD_OK;
        }
        if (mass_out) continue;                      // nothing to merge: the epilogue stored the probabilities
        if (lse)
            lmhead_merge_stats_kernel<<<(p.rows + 31) / 32, 256, 0, st>>>(p.part_key, p.part_idx, p.part_ref, p.part_sum,
                                                                           grid, p.rows, p.row0, p.c2, argmax, maxlogit, lse);
        else
            lmhead_merge_kernel<<<(p.rows + 127) / 128, 128, 0, st>>>(p.part_key, p.part_idx, grid, p.rows, p.row0,
                                                                     argmax, maxlogit);
        if (cudaGetLastError() != cudaSuccess) return SD_ERR_CUDA;
    }
    return SD_OK;
}

// probabilities of M rows over the whole vocabulary: mass[r][v] = exp(logit[r][v] * inv_temp - row_lse[r])
sd_status launch_lmhead_mass(const void* hidden, const void* W, int M, int Hd, int V, float inv_temp,
                             const float* row_lse, float* mass, void* ws, size_t ws_bytes,
                             int32_t* dev_status, cudaStream_t st) {
    return launch_lmhead_impl(hidden, W, M, Hd, V, nullptr, nullptr, ws, ws_bytes, dev_status, st, nullptr, inv_temp,
                              nullptr, mass, row_lse);
}

sd_status launch_lmhead_stats(const void* hidden, const void* W, int M, int Hd, int V, float inv_temp,
                              int32_t* argmax, float* maxlogit, float* lse, float* group_stats,
                              void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t st, float* logits) {
    return launch_lmhead_impl(hidden, W, M, Hd, V, argmax, maxlogit, ws, ws_bytes, dev_status, st, nullptr, inv_temp, lse,
                              nullptr, nullptr, group_stats, logits);
}

// only the tiles of the statistics pass (M <= 512): the caller's own kernel merges the per-CTA tables
sd_status launch_lmhead_stats_tiles(const void* hidden, const void* W, int M, int Hd, int V, float inv_temp,
                                    float* lse, float* group_stats, void* ws, size_t ws_bytes,
                                    int32_t* dev_status, cudaStream_t st, LmTables* tables) {
    int n_ctas = 0;
    const sd_status s = launch_lmhead_impl(hidden, W, M, Hd, V, nullptr, nullptr, ws, ws_bytes, dev_status, st, &n_ctas,
                                           inv_temp, lse, nullptr, nullptr, group_stats);
    if (s != SD_OK) return s;
    tables->part_key = static_cast<const int32_t*>(ws);
    tables->part_idx = tables->part_key + (size_t)kMaxCtas * kMaxCols;
    tables->part_ref = reinterpret_cast<const float*>(static_cast<const char*>(ws) + tail_workspace_bytes(M, V));
    tables->part_sum = tables->part_ref + (size_t)kMaxCtas * kMaxCols;
    tables->n_ctas = n_ctas;
    return SD_OK;
}

sd_status launch_lmhead(const void* hidden, const void* W, int M, int Hd, int V,
                        int32_t* argmax, float* maxlogit, void* ws, size_t ws_bytes,
                        int32_t* dev_status, cudaStream_t st) {
    return launch_lmhead_impl(hidden, W, M, Hd, V, argmax, maxlogit, ws, ws_bytes, dev_status, st, nullptr);
}

// ---------------------------------------------------------------------------
// Fused tail of a verify step.  CTA (b, l) merges the LM-head candidates of sequence b's rows
// (row = b * T_max + node), runs greedy acceptance on the resulting arg-max, and copies the
// accepted nodes' K/V into the cache of layer l.  The merge and the acceptance are a few
// microseconds of latency-bound work, so every layer's CTA repeats them rather than waiting for
// another CTA's result; only the CTAs of layer 0 write the arg-max and acceptance outputs.
// Replaces three launches (candidate merge, acceptance, compaction).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
tail_kernel(sd_batch bt, const __grid_constant__ CompactLayers ly,
            const int32_t* __restrict__ part_key, const int32_t* __restrict__ part_idx, int n_ctas,
            const int32_t* __restrict__ draft, int32_t* __restrict__ argmax, float* __restrict__ maxlogit,
            int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len, int32_t* status,
            int32_t* scratch /* [B][4 * T_max + 2]: outputs of the CTAs that must not write the real ones */) {
    __shared__ int32_t s_target[kMaxT];
    __shared__ int32_t s_path[kMaxT];
    __shared__ int s_na;
    const int b = blockIdx.x;
    const int layer = blockIdx.y;
    const int T = bt.T_max;
    const bool writer = (layer == 0);
    // 1. arg-max of this sequence's rows: eight threads per row, each an eighth of the CTAs' candidates
    for (int row0 = 0; row0 < T; row0 += 32) {
        const int row = row0 + (threadIdx.x >> 3), sub = threadIdx.x & 7;
        int32_t k = INT32_MIN, i = 0x7fffffff;
        if (row < T) {
            const int col = b * T + row;
#pragma unroll 4
            for (int c = sub; c < n_ctas; c += 8)
                take_better(k, i, __ldg(part_key + (size_t)c * kMaxCols + col), __ldg(part_idx + (size_t)c * kMaxCols + col));
        }
#pragma unroll
        for (int d = 1; d <= 4; d <<= 1) {
            const int32_t k2 = __shfl_xor_sync(0xffffffffu, k, d), i2 = __shfl_xor_sync(0xffffffffu, i, d);
            take_better(k, i, k2, i2);
        }
        if (row < T && sub == 0) {
            if (writer) {
                argmax[b * T + row] = i;
                if (maxlogit) maxlogit[b * T + row] = key_to_float(k);
            }
            s_target[row] = i;
        }
    }
    if (threadIdx.x == 0) s_na = 0;
    __syncthreads();
    // 2. greedy acceptance (one warp); CTAs of other layers keep their copy of the outputs to themselves
    if (threadIdx.x < 32) {
        int32_t* priv = scratch + ((size_t)blockIdx.y * gridDim.x) * (2 * T + 2);   // this layer's private area
        int32_t* o_nacc = writer ? n_acc : priv;                        // [B]
        int32_t* o_newlen = writer ? new_len : priv + gridDim.x;        // [B]
        int32_t* o_path = writer ? path : priv + 2 * gridDim.x;         // [B][T]
        int32_t* o_tok = writer ? out_tok : priv + 2 * gridDim.x + (size_t)gridDim.x * T;
        const int na = accept_sequence(bt, b, threadIdx.x, bt.parents + (size_t)b * T, draft + (size_t)b * T,
                                       s_target, o_nacc, o_path, o_tok, o_newlen, s_path, status);
        if (threadIdx.x == 0) s_na = na;
    }
    __syncthreads();
    // 3. accepted rows into this layer's cache
    compact_sequence(bt, ly, layer, 1, b, s_na, s_path, threadIdx.x, blockDim.x, status);
}

sd_status launch_lmhead_accept_compact(const sd_batch& bt, const void* hidden, const void* W, int Hd, int V,
                                       const int32_t* draft, const sd_kv_layer* layers, int L,
                                       const void* const* kt, const void* const* vt,
                                       int32_t* argmax, float* maxlogit, int32_t* n_acc, int32_t* path,
                                       int32_t* out_tok, int32_t* new_len, void* ws, size_t ws_bytes,
                                       int32_t* dev_status, cudaStream_t st) {
    const int M = bt.B * bt.T_max;
    if (M > kMaxCols || L > kLayersPerLaunch) {
        // shapes beyond one pass of the candidate tables or one set of layer descriptors: the same
        // three steps as separate launches
        sd_status s = launch_lmhead(hidden, W, M, Hd, V, argmax, maxlogit, ws, ws_bytes, dev_status, st);
        if (s != SD_OK) return s;
        s = launch_accept(bt, draft, argmax, n_acc, path, out_tok, new_len, dev_status, st);
        if (s != SD_OK) return s;
        return launch_compact(bt, layers, L, kt, vt, n_acc, path, dev_status, st);
    }
    if (ws_bytes < tail_workspace_bytes(M, V)) return SD_ERR_WORKSPACE;
    int n_ctas = 0;
    sd_status s = launch_lmhead_impl(hidden, W, M, Hd, V, argmax, maxlogit, ws, ws_bytes, dev_status, st, &n_ctas);
    if (s != SD_OK) return s;
    CompactLayers ly;
    fill_compact_layers(&ly, layers, kt, vt, 0, L);
    const int32_t* part_key = static_cast<const int32_t*>(ws);
    const int32_t* part_idx = part_key + (size_t)kMaxCtas * kMaxCols;
    // scratch for the non-writing CTAs' acceptance outputs: behind the candidate tables
    int32_t* scratch = static_cast<int32_t*>(ws) + (size_t)kMaxCtas * kMaxCols * 2;
    tail_kernel<<<dim3(bt.B, L), 256, 0, st>>>(bt, ly, part_key, part_idx, n_ctas, draft, argmax, maxlogit,
                                               n_acc, path, out_tok, new_len, dev_status, scratch);
    return cuda_ok(cudaGetLastError());
}


// ---------------------------------------------------------------------------
// Variant that needs no caller-provided scratch: the per-CTA candidate table
// lives in a fixed array inside the library image (1 MiB on every GPU that
// loads the library, held until the process exits).
// ---------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = (size_t)kMaxCtas * kMaxCols * 2 * sizeof(int32_t);
static __device__ __align__(256) unsigned char g_lmhead_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static std::atomic<void*> g_scratch_addr[kMaxDevices];     // device address of the array, per device ordinal

// The array's name is only a host-side handle here; the device address has to be
// asked for, once per device, with that device current.
static sd_status static_scratch(void** ptr) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SD_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return SD_ERR_UNSUPPORTED;
    void* p = g_scratch_addr[dev].load(std::memory_order_relaxed);
    if (!p) {
        // (two threads that both find the slot empty look the same address up twice: harmless)
        if (cudaGetSymbolAddress(&p, g_lmhead_scratch) != cudaSuccess || !p) return SD_ERR_CUDA;
        g_scratch_addr[dev].store(p, std::memory_order_relaxed);
    }
    *ptr = p;
    return SD_OK;
}

}  // namespace sdv

extern "C" sd_status sd_lmhead_argmax_static(const void* hidden, const void* W,
                                             int32_t M, int32_t Hd, int32_t V,
                                             int32_t* argmax, float* maxlogit,
                                             int32_t* dev_status, void* stream) {
    using namespace sdv;
    if (!hidden || !W || !argmax || !dev_status) return SD_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(W)) return SD_ERR_INVALID_ARG;
    if (M < 1 || V < 1 || Hd < 1) return SD_ERR_INVALID_ARG;
    if (Hd % 64 != 0) return SD_ERR_UNSUPPORTED;
    if (M > SD_LMHEAD_STATIC_MAX_ROWS) return SD_ERR_UNSUPPORTED;   // the built-in table holds one pass of rows
    void* scratch = nullptr;
    sd_status s = static_scratch(&scratch);
    if (s != SD_OK) return s;
    // Nothing in the table has to start at zero: every entry the merge reads is
    // written by this call's own CTAs first.
    return launch_lmhead(hidden, W, M, Hd, V, argmax, maxlogit, scratch, kStaticScratchBytes, dev_status,
                         static_cast<cudaStream_t>(stream));
}
