// Host-side declarations shared by the translation units of libac (not part of the public ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "ac.h"

namespace ac {

constexpr int kMaxDevices = 64;
// Fused merge inside a thread-block cluster: used when a (request, KV head)'s splits number at most
// this many and the grid has no more CTAs than the GPU has SMs (the plan prices it accordingly).
constexpr int kClusterMergeMaxSplits = 16;

struct DeviceState {
    bool ready = false;
    int sm_count = 0;
    int smem_optin = 0;
};

// Filled by ac_init; indexed by CUDA device ordinal.
DeviceState& device_state(int device);

// Records the CUDA error of the calling thread's last failure and returns AC_ERR_CUDA.
int fail_cuda(int code);

// Tokens per split for (max_context_len, num_splits): smallest multiple of 64 that covers it.
int split_tokens_for(int max_context_len, int num_splits);

struct CacheView {
    const void* k_cache;
    const void* v_cache;
    int64_t stride_page, stride_token, stride_head;   // elements
    int num_pages, page_size, Hkv, d;
};

// Prelude variants of the RoPE + append kernel and of the fused step (validated by the ABI layer).
struct RopeVariant {
    int rotary_dim;               // even, 2 .. d
    int interleaved;              // 0: pair (i, i + rotary_dim/2); 1: pair (2i, 2i + 1)
    const void* q_norm_weight;    // bf16 [d] or nullptr
    const void* k_norm_weight;    // bf16 [d] or nullptr
    float norm_eps;
};

// Extra inputs of the fused step: the attention kernel itself rotates q/k and appends k/v.
struct FusedRopeArgs {
    void* q_rot_out;          // optional
    const void* k_new;
    const void* v_new;
    void* k_cache;
    void* v_cache;
    int64_t stride_page, stride_token, stride_head;
    const float* rope_cos;
    const float* rope_sin;
    int max_position, num_pages;
    void* out_mirror;         // optional: a second copy of the bf16 result, e.g. in host memory the GPU can write
    const RopeVariant* variant;   // optional: prelude variants applied to q and k_new (nullptr: plain rotation)
};

// Per-kernel launchers; each validates nothing (the ABI layer did) and returns a cudaError_t.
cudaError_t attn_set_attributes(int smem_optin);
cudaError_t launch_rope_kv_append(const void* q_in, void* q_out, const void* k_new, const void* v_new,
                                  void* k_cache, void* v_cache, int64_t stride_page,
                                  int64_t stride_token, int64_t stride_head,
                                  const int32_t* block_table, int max_pages_per_seq,
                                  const int32_t* context_lens, const float* rope_cos,
                                  const float* rope_sin, int max_position, int B, int Hq, int Hkv,
                                  int d, int page_size, int num_pages, int32_t* status_flag,
                                  const RopeVariant* variant, cudaStream_t stream);
cudaError_t launch_paged_decode_attn(const CUtensorMap& k_map, const CUtensorMap& v_map,
                                     const void* q_rot,
                                     const int32_t* block_table, int max_pages_per_seq,
                                     const int32_t* context_lens, int new_tokens, float scale,
                                     int num_splits, int split_tokens, float* partial_o,
                                     float* partial_lse, int32_t* arrivals, void* out, int B, int Hq,
                                     int Hkv, int d, int page_size, int32_t* status_flag,
                                     const FusedRopeArgs* rope, int window, const int32_t* row_order,
                                     cudaStream_t stream);
cudaError_t qkv_set_attributes(int smem_optin);
int qkv_batch_tile(int B);
cudaError_t launch_qkv_rope_kv_append(const CUtensorMap& w_map, const CUtensorMap& x_map, void* q_out,
                                      void* k_cache, void* v_cache, int64_t stride_page,
                                      int64_t stride_token, int64_t stride_head,
                                      const int32_t* block_table, int max_pages_per_seq,
                                      const int32_t* context_lens, const float* rope_cos,
                                      const float* rope_sin, int max_position, int B, int H, int Hq,
                                      int Hkv, int d, int page_size, int num_pages, int32_t* status_flag,
                                      const RopeVariant* variant, cudaStream_t stream);
cudaError_t launch_oproj_residual(const CUtensorMap& w_map, const CUtensorMap& x_map,
                                  const void* residual_in, void* residual_out, int B, int K, int N,
                                  cudaStream_t stream);
cudaError_t launch_rmsnorm_rows(const void* h, const void* weight, void* out, int B, int N, float eps,
                                cudaStream_t stream);
cudaError_t proj_tc_set_attributes(int smem_optin);
int proj_tc_batch_rows(int B);          // rows of the x box the tcgen05 kernels expect for batch B
int proj_tc_k_blocks(int B);            // 64-element K blocks per TMA box (x and W) they expect for batch B
cudaError_t launch_qkv_rope_kv_append_tc(const CUtensorMap& w_map, const CUtensorMap& x_map, void* q_out,
                                         void* k_cache, void* v_cache, int64_t stride_page,
                                         int64_t stride_token, int64_t stride_head,
                                         const int32_t* block_table, int max_pages_per_seq,
                                         const int32_t* context_lens, const float* rope_cos,
                                         const float* rope_sin, int max_position, int B, int K, int Hq,
                                         int Hkv, int d, int page_size, int num_pages,
                                         int32_t* status_flag, const RopeVariant* variant, cudaStream_t stream);
cudaError_t launch_oproj_residual_tc(const CUtensorMap& w_map, const CUtensorMap& x_map,
                                     const void* residual_in, void* residual_out, int B, int K, int N,
                                     cudaStream_t stream);
cudaError_t launch_stage_inputs(const void* const src[5], void* const dst[5], const size_t bytes[5],
                                void* zero_dst, size_t zero_bytes, cudaStream_t stream);
cudaError_t launch_splitkv_merge(const float* partial_o, const float* partial_lse, int num_splits,
                                 const int32_t* context_lens, void* out, int B, int Hq, int d,
                                 cudaStream_t stream);

}  // namespace ac
