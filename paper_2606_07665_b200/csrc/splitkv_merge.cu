// A5: log-sum-exp merge of the per-split partial attention results.
//
// One CTA per (request, query head), one thread per 4 consecutive head_dim elements (16-byte loads of
// the fp32 partials).  Each thread first reduces the split log-sum-exps to their maximum M, then
// accumulates sum_s exp(lse_s - M) * partial_o[s] and the weight sum, and stores bf16.
#include <math.h>

#include "ac_device.cuh"
#include "ac_internal.h"

namespace ac {
namespace {

template <int D>
__global__ void __launch_bounds__(D / 4) splitkv_merge_kernel(
    const float* __restrict__ partial_o, const float* __restrict__ partial_lse, int num_splits,
    const int32_t* __restrict__ context_lens, uint16_t* __restrict__ out, int Hq) {
    const int hq = blockIdx.x;
    const int b = blockIdx.y;
    const size_t row = static_cast<size_t>(b) * Hq + hq;
    const int col = threadIdx.x * 4;
    uint2* dst = reinterpret_cast<uint2*>(out + row * D + col);
    const bool active = context_lens == nullptr || context_lens[b] >= 0;
    const float* lse = partial_lse + row * num_splits;
    float M = -INFINITY;
    if (active)
        for (int s = 0; s < num_splits; ++s) M = fmaxf(M, lse[s]);
    if (!(M > -INFINITY)) {            // inactive row, or every split empty
        *dst = make_uint2(0u, 0u);
        return;
    }
    const float4* po = reinterpret_cast<const float4*>(partial_o + row * num_splits * D + col);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    for (int s = 0; s < num_splits; ++s) {
        const float l = lse[s];
        if (l == -INFINITY) continue;                 // empty split: its partial_o is not valid
        const float w = __expf(l - M);
        const float4 v = po[static_cast<size_t>(s) * (D / 4)];
        acc.x = fmaf(w, v.x, acc.x);
        acc.y = fmaf(w, v.y, acc.y);
        acc.z = fmaf(w, v.z, acc.z);
        acc.w = fmaf(w, v.w, acc.w);
        den += w;
    }
    const float inv = 1.0f / den;
    *dst = make_uint2(acdev::pack_bf16x2(acc.x * inv, acc.y * inv),
                      acdev::pack_bf16x2(acc.z * inv, acc.w * inv));
}

}  // namespace

cudaError_t launch_splitkv_merge(const float* partial_o, const float* partial_lse, int num_splits,
                                 const int32_t* context_lens, void* out, int B, int Hq, int d,
                                 cudaStream_t stream) {
    dim3 grid(Hq, B);
    if (d == 128) {
        splitkv_merge_kernel<128><<<grid, 32, 0, stream>>>(partial_o, partial_lse, num_splits,
                                                           context_lens, static_cast<uint16_t*>(out), Hq);
    } else {
        splitkv_merge_kernel<64><<<grid, 16, 0, stream>>>(partial_o, partial_lse, num_splits,
                                                          context_lens, static_cast<uint16_t*>(out), Hq);
    }
    return cudaGetLastError();
}

}  // namespace ac
