// Shared device/host helpers of the sdverify kernels.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "sdverify.h"

namespace sdv {

constexpr int kBlock = 64;     // tokens per KV-cache block
constexpr int kD = 128;        // head dimension
constexpr int kMaxT = 64;      // nodes per tree

// first error wins; kernels never trap
__device__ __forceinline__ void set_status(int32_t* status, int code) {
    if (status) atomicCAS(status, 0, code);
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) {
    return __uint_as_float(((uint32_t)b) << 16);
}
__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline sd_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? SD_OK : SD_ERR_CUDA; }

// Test hooks, read from the environment at every launch (unset in normal use):
//   SDV_TEST_WAIT_CYCLES  bound of the kernels' barrier waits in SM cycles (default: about a second)
//   SDV_TEST_WITHHOLD     1: one role of the tensor-core kernels withholds its first arrival, so that
//                         a bounded wait runs out and the launch ends with SD_ERR_TIMEOUT
//   SDV_TEST_CHUNKS       1, 2, 4 or 8: key chunks per sequence of single-launch attention calls
struct TestKnobs { long long wait_cycles; int withhold; int chunks; };
TestKnobs test_knobs();

// launch-side entry points implemented in the kernel files
sd_status launch_tree_prepare(const sd_batch& bt, int32_t* dev_status, cudaStream_t st);
sd_status launch_accept(const sd_batch& bt, const int32_t* draft, const int32_t* target,
                        int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                        int32_t* dev_status, cudaStream_t st);
sd_status launch_compact(const sd_batch& bt, const sd_kv_layer* layers, int L,
                         const void* const* kt, const void* const* vt,
                         const int32_t* n_acc, const int32_t* path, int32_t* dev_status, cudaStream_t st);
size_t attention_workspace_bytes(const sd_batch& bt);
sd_status launch_attention(const sd_batch& bt, const sd_kv_layer& cache, const void* q,
                           const void* kt, const void* vt, float scale, void* out, float* lse,
                           void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t st);
sd_status launch_attention_layers(const sd_batch& bt, const sd_kv_layer* caches, int L,
                                  const void* const* q, const void* const* kt, const void* const* vt,
                                  float scale, void* const* out, float* const* lse,
                                  int32_t* dev_status, cudaStream_t st);
size_t lmhead_workspace_bytes(int M, int V);
size_t tail_workspace_bytes(int M, int V);
sd_status launch_lmhead(const void* hidden, const void* W, int M, int Hd, int V,
                        int32_t* argmax, float* maxlogit, void* ws, size_t ws_bytes,
                        int32_t* dev_status, cudaStream_t st);

sd_status launch_lmhead_accept_compact(const sd_batch& bt, const void* hidden, const void* W, int Hd, int V,
                                       const int32_t* draft, const sd_kv_layer* layers, int L,
                                       const void* const* kt, const void* const* vt,
                                       int32_t* argmax, float* maxlogit, int32_t* n_acc, int32_t* path,
                                       int32_t* out_tok, int32_t* new_len, void* ws, size_t ws_bytes,
                                       int32_t* dev_status, cudaStream_t st);

sd_status launch_draft_feature_attention(const void* qp, const void* k, const void* v, int S, int L, int Q, int H,
                                         float scale, void* out, cudaStream_t st);
size_t stats_workspace_bytes(int M, int V);
sd_status launch_lmhead_stats(const void* hidden, const void* W, int M, int Hd, int V, float inv_temp,
                              int32_t* argmax, float* maxlogit, float* lse, float* group_stats,
                              void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t st, float* logits = nullptr);
sd_status launch_lmhead_mass(const void* hidden, const void* W, int M, int Hd, int V, float inv_temp,
                             const float* row_lse, float* mass, void* ws, size_t ws_bytes,
                             int32_t* dev_status, cudaStream_t st);
// per-CTA tables the LM-head tiles of a statistics pass leave in the workspace (row stride 512 entries)
struct LmTables { const int32_t* part_key; const int32_t* part_idx; const float* part_ref; const float* part_sum; int n_ctas; };
sd_status launch_lmhead_stats_tiles(const void* hidden, const void* W, int M, int Hd, int V, float inv_temp,
                                    float* lse, float* group_stats, void* ws, size_t ws_bytes,
                                    int32_t* dev_status, cudaStream_t st, LmTables* tables);
size_t sampled_workspace_bytes(int B, int T, int V, int Hd);
sd_status launch_accept_sampled(const sd_batch& bt, const void* hidden, const void* W, int Hd, int V, float inv_temp,
                                const float* lse, const float* group_stats, const int32_t* draft, const float* u,
                                const float* w, int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                                void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t st);

sd_status launch_accept_chain_sampled(const sd_batch& bt, const void* hidden, const void* W, int Hd, int V, float inv_temp,
                                      const float* lse, const float* logits, const int32_t* draft, const float* q_tok,
                                      const float* q_rows, const float* u, const float* w, int32_t* n_acc, int32_t* path,
                                      int32_t* out_tok, int32_t* new_len, void* ws, size_t ws_bytes, int32_t* dev_status,
                                      cudaStream_t st);
sd_status launch_accept_tree_sampled_q(const sd_batch& bt, int V, float inv_temp, const float* lse, const float* logits,
                                       const int32_t* draft, const float* q_rows, const float* u, const float* w,
                                       int32_t* n_acc, int32_t* path, int32_t* out_tok, int32_t* new_len,
                                       int32_t* dev_status, cudaStream_t st);
sd_status launch_lmhead_accept_sampled_compact(const sd_batch& bt, const void* hidden, const void* W, int Hd, int V,
                                               float inv_temp, const int32_t* draft, const float* u, const float* w,
                                               const sd_kv_layer* layers, int L, const void* const* kt, const void* const* vt,
                                               float* lse, float* group_stats, int32_t* n_acc, int32_t* path,
                                               int32_t* out_tok, int32_t* new_len, void* ws, size_t ws_bytes,
                                               int32_t* dev_status, cudaStream_t st);

}  // namespace sdv
