// Split-KV decode attention + merge for callers that may not allocate device memory.
//
// The split partials normally live in a workspace the caller allocates.  Some callers cannot do
// that: a serving engine that handed every free byte of HBM to its KV-cache pool at start-up, a
// plug-in that runs while its host framework forbids cudaMalloc (a pool allocator with a fixed
// reservation, or a region of code that must not take the driver's allocation lock), or a step
// function that has no place to keep a buffer between calls.  For them this file keeps the
// partials in a fixed array that is part of the library image: every GPU that loads the library
// holds AC_STATIC_SCRATCH_BYTES of it until the process exits.
//
// In host code the array's name is only a handle: its device address is looked up once per device
// with cudaGetSymbolAddress (in this translation unit, which owns the array) and that address is
// what the kernels receive.
#include <math.h>

#include <mutex>

#include "ac_internal.h"

namespace ac {
namespace {

// Partials of one call: partial_o fp32 [B,Hq,S,d] followed by partial_lse fp32 [B,Hq,S].
static __device__ __align__(256) unsigned char g_static_scratch[AC_STATIC_SCRATCH_BYTES];

std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the array on the current device; resolved on the first call per device.
cudaError_t scratch_address(int device, void** out) {
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_addr[device] == nullptr) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (ptr == nullptr) return cudaErrorInvalidSymbol;
        g_scratch_addr[device] = ptr;
    }
    *out = g_scratch_addr[device];
    return cudaSuccess;
}

}  // namespace
}  // namespace ac

using namespace ac;

extern "C" int ac_paged_decode_attn_static_scratch(
    const void* q_rot, const void* k_cache, const void* v_cache, int64_t stride_page,
    int64_t stride_token, int64_t stride_head, const int32_t* block_table, int max_pages_per_seq,
    const int32_t* context_lens, int new_tokens, float softmax_scale, int num_splits, void* out, int B,
    int Hq, int Hkv, int d, int page_size, int num_pages, int max_context_len, int32_t* status_flag,
    void* stream) {
    // Every check that the two inner calls would make on `out`, B, Hq, d and num_splits is made here
    // first, so that an error can only come back before anything has been enqueued.
    if (!out) return AC_ERR_NULL;
    if (B <= 0 || Hq <= 0 || d <= 0 || num_splits <= 0) return AC_ERR_SHAPE;
    if (d != 64 && d != 128) return AC_ERR_UNSUPPORTED;
    if (B > 65535 || num_splits > 65535) return AC_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(out) & 15u) return AC_ERR_ALIGN;
    if (num_splits == 1) {
        // One split: the existing entry point writes the final rows to `out` directly and touches
        // no scratch at all, so the size limit does not apply.
        return ac_paged_decode_attn(q_rot, k_cache, v_cache, stride_page, stride_token, stride_head,
                                    block_table, max_pages_per_seq, context_lens, new_tokens,
                                    softmax_scale, 1, nullptr, 0, out, B, Hq, Hkv, d, page_size,
                                    num_pages, max_context_len, status_flag, stream);
    }
    const unsigned long long need = static_cast<unsigned long long>(B) * Hq * num_splits *
                                    (static_cast<unsigned long long>(d) + 1) * sizeof(float);
    if (need > AC_STATIC_SCRATCH_BYTES) return AC_ERR_SCRATCH_LIMIT;
    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return fail_cuda(static_cast<int>(e));
    if (device < 0 || device >= kMaxDevices) return AC_ERR_UNSUPPORTED;
    if (!device_state(device).ready) return AC_ERR_NOT_INIT;
    void* scratch = nullptr;
    e = scratch_address(device, &scratch);
    if (e != cudaSuccess) return fail_cuda(static_cast<int>(e));

    // Nothing in the array has to start at zero: every CTA of the attention kernel overwrites the
    // log-sum-exp slot of its own split (a number, or -inf for a split with no tokens) before the
    // merge reads it, and the merge never reads the partial_o of a split whose slot is -inf.  What
    // an earlier call left behind is therefore either overwritten or ignored.
    const int st = ac_paged_decode_attn(q_rot, k_cache, v_cache, stride_page, stride_token, stride_head,
                                        block_table, max_pages_per_seq, context_lens, new_tokens,
                                        softmax_scale, num_splits, scratch, static_cast<size_t>(need), out,
                                        B, Hq, Hkv, d, page_size, num_pages, max_context_len, status_flag,
                                        stream);
    if (st != AC_OK) return st;
    return ac_splitkv_merge(scratch, num_splits, context_lens, out, B, Hq, d, stream);
}
