// Staging of one decode step's host-resident inputs for ac_decode_step_host.
//
// The step's inputs (q, k_new, v_new, block_table, context_lens) are small (a few hundred KB) and
// live in pinned host memory that the GPU can address directly.  Five separate copy-engine
// transfers cost a few microseconds each of set-up latency on the stream; one kernel that reads all
// five buffers over the host link with many threads in flight, and clears the arrival counters of
// the fused merge on the way, takes about as long as a single one of them.
#include "ac_internal.h"

namespace ac {
namespace {

struct StageList {
    const uint4* src[5];
    uint4* dst[5];
    unsigned long long chunks[5];      // 16-byte pieces per buffer
    uint4* zero_dst;                   // region to clear (may be null)
    unsigned long long zero_chunks;
};

__global__ void __launch_bounds__(256) stage_inputs_kernel(const StageList list) {
    // No early launch-completion trigger here: the attention kernel that follows reads context_lens
    // and block_table (written by this kernel) BEFORE it synchronises on its predecessor, so it must
    // not become resident until this grid has finished.
    const unsigned long long tid = blockIdx.x * 256ull + threadIdx.x;
    const unsigned long long stride = gridDim.x * 256ull;
    // The five buffers are one index space: a thread's pieces come from whichever buffers they fall
    // in, so every read over the host link is in flight at once (one buffer after the other made the
    // threads that serve several buffers pay one link round trip per buffer).
    unsigned long long total = 0;
#pragma unroll
    for (int b = 0; b < 5; ++b) total += list.chunks[b];
    auto locate = [&](unsigned long long i, int& b, unsigned long long& k) {
        k = i;
        b = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (b == c && k >= list.chunks[c]) {
                k -= list.chunks[c];
                b = c + 1;
            }
    };
    // The host buffers are complete when the call is made; the device buffers may still be read by the
    // kernel ahead of this one.  So a thread's first piece crosses the host link BEFORE the wait for
    // that kernel (this grid becomes resident beside it under programmatic stream serialization) and is
    // stored after it.
    int b0 = 0;
    unsigned long long k0 = 0;
    uint4 first = make_uint4(0u, 0u, 0u, 0u);
    if (tid < total) {
        locate(tid, b0, k0);
        first = list.src[b0][k0];
    }
    cudaGridDependencySynchronize();
    if (tid < total) list.dst[b0][k0] = first;
    for (unsigned long long i = tid + stride; i < total; i += stride) {
        int b;
        unsigned long long k;
        locate(i, b, k);
        list.dst[b][k] = list.src[b][k];
    }
    for (unsigned long long i = tid; i < list.zero_chunks; i += stride)
        list.zero_dst[i] = make_uint4(0u, 0u, 0u, 0u);
}

}  // namespace

// All sizes in bytes and multiples of 16 except the last piece of each buffer, which the caller
// rounds up (device buffers from cudaMalloc-class allocators are padded well beyond 16 bytes; host
// sizes are checked by the caller).  Returns cudaErrorInvalidValue, having launched nothing, when a
// source is not device-addressable host memory or a size or address is not a multiple of 16.
cudaError_t launch_stage_inputs(const void* const src[5], void* const dst[5], const size_t bytes[5],
                                void* zero_dst, size_t zero_bytes, cudaStream_t stream) {
    StageList list;
    unsigned long long total = 0;
    for (int b = 0; b < 5; ++b) {
        if (bytes[b] % 16 != 0) return cudaErrorInvalidValue;
        cudaPointerAttributes attr;
        cudaError_t e = cudaPointerGetAttributes(&attr, src[b]);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return cudaErrorInvalidValue;
        }
        if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) return cudaErrorInvalidValue;
        if ((reinterpret_cast<uintptr_t>(attr.devicePointer) | reinterpret_cast<uintptr_t>(dst[b])) & 15u)
            return cudaErrorInvalidValue;                 // the kernel moves 16-byte pieces
        list.src[b] = static_cast<const uint4*>(attr.devicePointer);
        list.dst[b] = static_cast<uint4*>(dst[b]);
        list.chunks[b] = bytes[b] / 16;
        total += list.chunks[b];
    }
    if (zero_bytes % 16 != 0 || (reinterpret_cast<uintptr_t>(zero_dst) & 15u)) return cudaErrorInvalidValue;
    list.zero_dst = static_cast<uint4*>(zero_dst);
    list.zero_chunks = zero_dst != nullptr ? zero_bytes / 16 : 0;
    total += list.zero_chunks;
    unsigned blocks = static_cast<unsigned>((total + 255) / 256);
    if (blocks < 1) blocks = 1;
    if (blocks > 592) blocks = 592;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, stage_inputs_kernel, list);
}

}  // namespace ac
