// A1 + A2: rotary embedding of the new q/k and scatter of the new k/v into the paged cache.
//
// One thread handles 8 consecutive pair indices i..i+7 of one head vector: it loads 16 bytes from
// the first half of the vector and 16 bytes from the second half, 2 x 32 bytes of cos and sin,
// rotates in fp64 and stores 2 x 16 bytes.  Head vectors are numbered per request as
// [0, Hq) = query heads (written to q_out) and [Hq, Hq + Hkv) = KV heads (rotated k written to the
// cache slot, v copied verbatim to the same slot of the V pool).
//
// Rounding: every stored value is the nearest-even bf16 of the real number a*c -/+ b*s.  Both
// products are exact in fp64 (8-bit x 24-bit significands), the sum is one fp64 rounding, and the
// fp64 -> bf16 step goes through an fp32 obtained by round-to-odd, which makes the final
// round-to-nearest-even identical to a direct rounding of the fp64 value.
#include "ac_device.cuh"
#include "ac_internal.h"
#include "rope_variant.cuh"

namespace ac {
namespace {

struct alignas(16) Vec8 {
    uint16_t v[8];
};

template <int D>
__global__ void __launch_bounds__(128) rope_kv_append_kernel(
    const uint16_t* q_in, uint16_t* q_out,   // may alias (in-place rotation)
    const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
    uint16_t* __restrict__ k_cache, uint16_t* __restrict__ v_cache, int64_t stride_page,
    int64_t stride_token, int64_t stride_head, const int32_t* __restrict__ block_table,
    int max_pages_per_seq, const int32_t* __restrict__ context_lens,
    const float* __restrict__ rope_cos, const float* __restrict__ rope_sin, int max_position, int B,
    int Hq, int Hkv, int page_size, int num_pages, int32_t* status_flag) {
    // This kernel may have been launched early, under the tail of the previous attention kernel, whose
    // inputs (the rotated q buffer, the cache) it overwrites: wait for that kernel first.  Only then
    // is the dependent kernel (the attention launch that follows) let in to begin its own set-up; it
    // synchronises on this grid's completion before reading anything written here.  Signalling after
    // the wait keeps a chain of launches at most two kernels deep, which is what the attention
    // kernel's early tile loads rely on.
    cudaGridDependencySynchronize();
    cudaTriggerProgrammaticLaunchCompletion();
    constexpr int HALF = D / 2;
    constexpr int THREADS_PER_VEC = HALF / 8;            // 8 (D=128) or 4 (D=64)
    const int heads = Hq + Hkv;
    const long long gid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long long vec = gid / THREADS_PER_VEC;
    const int i0 = static_cast<int>(gid % THREADS_PER_VEC) * 8;
    if (vec >= static_cast<long long>(B) * heads) return;
    const int b = static_cast<int>(vec / heads);
    const int hh = static_cast<int>(vec % heads);
    const int p = context_lens[b];
    if (p < 0) return;                                    // inactive row
    const int page_idx = p / page_size;
    if (p >= max_position || page_idx >= max_pages_per_seq) {
        if (status_flag != nullptr && i0 == 0) atomicOr(status_flag, AC_FLAG_POSITION_OOB);
        return;
    }

    const bool is_q = hh < Hq;
    const uint16_t* src;
    uint16_t* dst;
    uint16_t* dst_v = nullptr;
    const uint16_t* src_v = nullptr;
    if (is_q) {
        src = q_in + (static_cast<size_t>(b) * Hq + hh) * D;
        dst = q_out + (static_cast<size_t>(b) * Hq + hh) * D;
    } else {
        const int h = hh - Hq;
        const int page = block_table[static_cast<size_t>(b) * max_pages_per_seq + page_idx];
        if (page < 0 || page >= num_pages) {
            if (status_flag != nullptr && i0 == 0) atomicOr(status_flag, AC_FLAG_PAGE_OOB);
            return;
        }
        const int slot = p - page_idx * page_size;
        const size_t off = static_cast<size_t>(page) * stride_page +
                           static_cast<size_t>(slot) * stride_token +
                           static_cast<size_t>(h) * stride_head;
        src = k_new + (static_cast<size_t>(b) * Hkv + h) * D;
        dst = k_cache + off;
        src_v = v_new + (static_cast<size_t>(b) * Hkv + h) * D;
        dst_v = v_cache + off;
    }

    const Vec8 lo = *reinterpret_cast<const Vec8*>(src + i0);
    const Vec8 hi = *reinterpret_cast<const Vec8*>(src + HALF + i0);
    const float4* cp = reinterpret_cast<const float4*>(rope_cos + static_cast<size_t>(p) * HALF + i0);
    const float4* sp = reinterpret_cast<const float4*>(rope_sin + static_cast<size_t>(p) * HALF + i0);
    const float4 c0 = cp[0], c1 = cp[1], s0 = sp[0], s1 = sp[1];
    const float c[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
    const float s[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
    Vec8 out_lo, out_hi;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        out_lo.v[e] = acdev::rope_first_half(lo.v[e], hi.v[e], c[e], s[e]);
        out_hi.v[e] = acdev::rope_second_half(lo.v[e], hi.v[e], c[e], s[e]);
    }
    *reinterpret_cast<Vec8*>(dst + i0) = out_lo;
    *reinterpret_cast<Vec8*>(dst + HALF + i0) = out_hi;
    if (!is_q) {
        // v is copied verbatim: this thread moves the same two 16-byte pieces of the v vector.
        *reinterpret_cast<Vec8*>(dst_v + i0) = *reinterpret_cast<const Vec8*>(src_v + i0);
        *reinterpret_cast<Vec8*>(dst_v + HALF + i0) = *reinterpret_cast<const Vec8*>(src_v + HALF + i0);
    }
}


// Variants of the prelude (per-head RMSNorm of q/k before the rotation, partial rotary, interleaved
// pairing): one warp per head vector.  The (optionally normalised) vector is parked in shared memory
// so that every lane can read the partner of each of its elements, wherever the pairing puts it.
//
// RMSNorm arithmetic: sum of squares in fp64 (exact for bf16 inputs of moderate dynamic range),
// r = 1 / sqrt(sum / d + eps) with correctly rounded fp64 sqrt and division, y = bf16(x * r), then
// bf16(y * w): normalise, round to the model dtype, scale by the weight, round again.
template <int D>
__global__ void __launch_bounds__(128) rope_kv_append_ex_kernel(
    const uint16_t* q_in, uint16_t* q_out, const uint16_t* __restrict__ k_new,
    const uint16_t* __restrict__ v_new, uint16_t* __restrict__ k_cache, uint16_t* __restrict__ v_cache,
    int64_t stride_page, int64_t stride_token, int64_t stride_head,
    const int32_t* __restrict__ block_table, int max_pages_per_seq,
    const int32_t* __restrict__ context_lens, const float* __restrict__ rope_cos,
    const float* __restrict__ rope_sin, int max_position, int B, int Hq, int Hkv, int page_size,
    int num_pages, int32_t* status_flag, int rotary_dim, int interleaved,
    const uint16_t* __restrict__ q_norm_w, const uint16_t* __restrict__ k_norm_w, float norm_eps) {
    cudaGridDependencySynchronize();               // as in the plain kernel: wait, then let the next one in
    cudaTriggerProgrammaticLaunchCompletion();
    constexpr int EPL = D / 32;                           // elements per lane: 4 (D=128) or 2 (D=64)
    __shared__ uint16_t s_vec[4][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int heads = Hq + Hkv;
    const long long vec = static_cast<long long>(blockIdx.x) * 4 + warp;
    if (vec >= static_cast<long long>(B) * heads) return;
    const int b = static_cast<int>(vec / heads);
    const int hh = static_cast<int>(vec % heads);
    const int p = context_lens[b];
    if (p < 0) return;
    const int page_idx = p / page_size;
    if (p >= max_position || page_idx >= max_pages_per_seq) {
        if (status_flag != nullptr && lane == 0) atomicOr(status_flag, AC_FLAG_POSITION_OOB);
        return;
    }
    const bool is_q = hh < Hq;
    const uint16_t* src;
    uint16_t* dst;
    const uint16_t* norm_w;
    size_t cache_off = 0;
    if (is_q) {
        src = q_in + (static_cast<size_t>(b) * Hq + hh) * D;
        dst = q_out + (static_cast<size_t>(b) * Hq + hh) * D;
        norm_w = q_norm_w;
    } else {
        const int h = hh - Hq;
        const int page = block_table[static_cast<size_t>(b) * max_pages_per_seq + page_idx];
        if (page < 0 || page >= num_pages) {
            if (status_flag != nullptr && lane == 0) atomicOr(status_flag, AC_FLAG_PAGE_OOB);
            return;
        }
        cache_off = static_cast<size_t>(page) * stride_page +
                    static_cast<size_t>(p - page_idx * page_size) * stride_token +
                    static_cast<size_t>(h) * stride_head;
        src = k_new + (static_cast<size_t>(b) * Hkv + h) * D;
        dst = k_cache + cache_off;
        norm_w = k_norm_w;
    }

    uint16_t x[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) x[e] = src[lane * EPL + e];
    acdev::rope_variant_vector<D>(x, norm_w, norm_eps, rope_cos + static_cast<size_t>(p) * (rotary_dim / 2),
                                  rope_sin + static_cast<size_t>(p) * (rotary_dim / 2), rotary_dim, interleaved,
                                  s_vec[warp], lane);
#pragma unroll
    for (int e = 0; e < EPL; ++e) dst[lane * EPL + e] = x[e];
    if (!is_q) {
        const uint16_t* src_v = v_new + (static_cast<size_t>(b) * Hkv + (hh - Hq)) * D;
#pragma unroll
        for (int e = 0; e < EPL; ++e) v_cache[cache_off + lane * EPL + e] = src_v[lane * EPL + e];
    }
}

}  // namespace

cudaError_t launch_rope_kv_append(const void* q_in, void* q_out, const void* k_new, const void* v_new,
                                  void* k_cache, void* v_cache, int64_t stride_page,
                                  int64_t stride_token, int64_t stride_head,
                                  const int32_t* block_table, int max_pages_per_seq,
                                  const int32_t* context_lens, const float* rope_cos,
                                  const float* rope_sin, int max_position, int B, int Hq, int Hkv,
                                  int d, int page_size, int num_pages, int32_t* status_flag,
                                  const RopeVariant* variant, cudaStream_t stream) {
    if (variant != nullptr) {
        cudaLaunchConfig_t cfg = {};
        const long long vecs = static_cast<long long>(B) * (Hq + Hkv);
        cfg.gridDim = dim3(static_cast<unsigned>((vecs + 3) / 4));
        cfg.blockDim = dim3(128);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
#define AC_ROPE_EX_ARGS                                                                           \
    static_cast<const uint16_t*>(q_in), static_cast<uint16_t*>(q_out),                             \
        static_cast<const uint16_t*>(k_new), static_cast<const uint16_t*>(v_new),                  \
        static_cast<uint16_t*>(k_cache), static_cast<uint16_t*>(v_cache), stride_page,             \
        stride_token, stride_head, block_table, max_pages_per_seq, context_lens, rope_cos,         \
        rope_sin, max_position, B, Hq, Hkv, page_size, num_pages, status_flag,                     \
        variant->rotary_dim, variant->interleaved,                                                 \
        static_cast<const uint16_t*>(variant->q_norm_weight),                                      \
        static_cast<const uint16_t*>(variant->k_norm_weight), variant->norm_eps
        if (d == 128) return cudaLaunchKernelEx(&cfg, rope_kv_append_ex_kernel<128>, AC_ROPE_EX_ARGS);
        return cudaLaunchKernelEx(&cfg, rope_kv_append_ex_kernel<64>, AC_ROPE_EX_ARGS);
#undef AC_ROPE_EX_ARGS
    }
    const long long threads_per_vec = d / 16;
    const long long total = static_cast<long long>(B) * (Hq + Hkv) * threads_per_vec;
    const int block = 128;
    const unsigned grid = static_cast<unsigned>((total + block - 1) / block);
#define AC_ROPE_ARGS                                                                              \
    static_cast<const uint16_t*>(q_in), static_cast<uint16_t*>(q_out),                             \
        static_cast<const uint16_t*>(k_new), static_cast<const uint16_t*>(v_new),                  \
        static_cast<uint16_t*>(k_cache), static_cast<uint16_t*>(v_cache), stride_page,             \
        stride_token, stride_head, block_table, max_pages_per_seq, context_lens, rope_cos,         \
        rope_sin, max_position, B, Hq, Hkv, page_size, num_pages, status_flag
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (d == 128) {
        e = cudaLaunchKernelEx(&cfg, rope_kv_append_kernel<128>, AC_ROPE_ARGS);
    } else {
        e = cudaLaunchKernelEx(&cfg, rope_kv_append_kernel<64>, AC_ROPE_ARGS);
    }
#undef AC_ROPE_ARGS
    return e;
}

}  // namespace ac
