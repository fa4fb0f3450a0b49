// Device-side helpers shared by the kernels of libac: PTX wrappers for shared-memory barriers,
// tensor-map (TMA) tile loads, ldmatrix, the bf16 warp MMA, and bf16 packing.  sm_100a only.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace acdev {

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier -------------------------------------------------------------------------------

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(arrivals) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Makes freshly initialised barriers visible to the async (TMA) proxy.
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Orders this thread's earlier ordinary stores to shared memory before later accesses to the same
// bytes through the async proxy (a TMA load that overwrites them).
__device__ __forceinline__ void fence_proxy_async_shared() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done != 0;
}

// Waits for the phase with the given parity to complete, for at most ~2^31 SM cycles (about a
// second).  Returns false when it gave up; the caller records that and stops consuming the buffer.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > (1ll << 31)) return false;
    }
    return true;
}

// ---- TMA: 5-D tiled load global -> shared of this CTA, completion counted on an mbarrier --------

__device__ __forceinline__ void tma_prefetch_descriptor(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// L2 eviction policy for data that is read exactly once.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// L2 eviction policy for data that every CTA of the grid reads again.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        ".L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2),
        "l"(policy)
        : "memory");
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3, int c4, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        ".L2::cache_hint [%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2),
        "r"(c3), "r"(c4), "l"(policy)
        : "memory");
}

// ---- thread-block clusters: distributed shared memory ----------------------------------------------

// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t cluster_map_shared(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float4 cluster_load_f32x4(uint32_t cluster_addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(cluster_addr)
                 : "memory");
    return v;
}
__device__ __forceinline__ float cluster_load_f32(uint32_t cluster_addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(cluster_addr) : "memory");
    return v;
}
__device__ __forceinline__ double cluster_load_f64(uint32_t cluster_addr) {
    double v;
    asm volatile("ld.shared::cluster.f64 %0, [%1];" : "=d"(v) : "r"(cluster_addr) : "memory");
    return v;
}
__device__ __forceinline__ uint16_t cluster_load_u16(uint32_t cluster_addr) {
    uint16_t v;
    asm volatile("ld.shared::cluster.u16 %0, [%1];" : "=h"(v) : "r"(cluster_addr) : "memory");
    return v;
}
// Hardware barrier over the threads of the cluster (not a spin); every CTA of the cluster must execute
// the same number of them on every path.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// The two halves of that barrier, for a CTA that only has to outlive its sisters' reads of its shared
// memory: arrive when done reading theirs, wait before exiting.  No other cluster barrier in between.
__device__ __forceinline__ void cluster_arrive_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
// Arrival that publishes nothing (a pure "I am done with your shared memory"): it does not wait for the
// thread's earlier stores to become visible, as the releasing form does.
__device__ __forceinline__ void cluster_arrive_relaxed_all() {
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait_all() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// ---- ldmatrix / mma ---------------------------------------------------------------------------

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                            uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr)
                 : "memory");
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr)
                 : "memory");
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col).  Rows 0-7 of the tile are c0,c1 / a0,a2;
// rows 8-15 are c2,c3 / a1,a3.
__device__ __forceinline__ void mma_bf16_16816(float& c0, float& c1, float& c2, float& c3,
                                               uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
        "{%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3)
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Same product when only rows 0-7 of A are populated: rows 8-15 of the result are discarded.
__device__ __forceinline__ void mma_bf16_16816_top(float& c0, float& c1, uint32_t a0, uint32_t a2,
                                                   uint32_t b0, uint32_t b1) {
    float d2, d3;
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
        "{%8, %9}, {%0, %1, %10, %10};"
        : "+f"(c0), "+f"(c1), "=f"(d2), "=f"(d3)
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1), "f"(0.0f));
    (void)d2;
    (void)d3;
}

// ---- bf16 packing -----------------------------------------------------------------------------

// (lo, hi) fp32 -> two round-to-nearest-even bf16 in one 32-bit word, lo in the low half.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) {
    return __uint_as_float(static_cast<uint32_t>(b) << 16);
}

// ---- rotary embedding of one pair, exact then rounded once ------------------------------------

// Nearest-even bf16 of an fp64 value without double rounding: fp64 -> fp32 by truncation with a
// sticky bit (round to odd), then the usual nearest-even cut to 16 bits.
__device__ __forceinline__ uint16_t f64_to_bf16_rne(double x) {
    float f = __double2float_rz(x);
    uint32_t u = __float_as_uint(f);
    if (static_cast<double>(f) != x) u |= 1u;          // sticky bit: round to odd (NaN stays NaN)
    if ((u & 0x7F800000u) == 0x7F800000u) {            // inf or NaN
        return static_cast<uint16_t>((u >> 16) | ((u & 0xFFFFu) ? 0x40u : 0u));
    }
    u += 0x7FFFu + ((u >> 16) & 1u);
    return static_cast<uint16_t>(u >> 16);
}

// (a, b) = (x_i, x_{i+d/2}) as bf16 bits, c/s = cos/sin of the pair's angle.  Both products are exact
// in fp64 (8-bit x 24-bit significands); __dmul_rn/__dadd_rn keep the three operations separate.
__device__ __forceinline__ uint16_t rope_first_half(uint16_t a, uint16_t b, float c, float s) {
    const double ad = static_cast<double>(bf16_bits_to_float(a));
    const double bd = static_cast<double>(bf16_bits_to_float(b));
    return f64_to_bf16_rne(__dsub_rn(__dmul_rn(ad, static_cast<double>(c)), __dmul_rn(bd, static_cast<double>(s))));
}

__device__ __forceinline__ uint16_t rope_second_half(uint16_t a, uint16_t b, float c, float s) {
    const double ad = static_cast<double>(bf16_bits_to_float(a));
    const double bd = static_cast<double>(bf16_bits_to_float(b));
    return f64_to_bf16_rne(__dadd_rn(__dmul_rn(bd, static_cast<double>(c)), __dmul_rn(ad, static_cast<double>(s))));
}

// ---- the same rotation for callers that rotate thousands of values per CTA ------------------------
//
// bf16_rne(fl64(x1 * y1 - x2 * y2)) for x1, x2 with bf16 precision (8-bit significands) and fp32 y1, y2
// is what the two functions above compute (first half: a c - b s; second half: b c - a (-s)).  That
// evaluation costs a dozen fp64-pipe instructions per output, which a kernel that rotates a few
// values per thread never notices and an epilogue that rotates 128 rows x 48 features does.  The
// fp32 evaluation below gives the same bits whenever it can prove so: error-free products (product and
// fma residual), an error-free difference of the high parts (TwoSum), and the small terms added on
// top give r with |r - exact| < 0.501 ulp(r) provided the difference did not cancel more than ten bits
// and nothing is near the fp32 range limits.  If r is then at least three fp32 ulps away from every
// midpoint between adjacent bf16 values (low half-word not in 0x7FFE..0x8002), the exact value, its
// fp64 rounding and r all round to the same bf16.  Callers evaluate a batch without branches and
// repair the (rare) unproven ones afterwards with rope_diff_of_products_f64.
__device__ __forceinline__ uint16_t rope_diff_of_products_f32(float x1, float y1, float x2, float y2, bool& proven) {
    const float p1 = __fmul_rn(x1, y1);
    const float p1l = __fmaf_rn(x1, y1, -p1);            // exact: the product has at most 32 bits
    const float p2 = __fmul_rn(x2, y2);
    const float p2l = __fmaf_rn(x2, y2, -p2);
    const float sh = __fsub_rn(p1, p2);
    const float bv = __fsub_rn(sh, p1);
    const float e = __fadd_rn(__fsub_rn(p1, __fsub_rn(sh, bv)), __fsub_rn(-p2, bv));   // sh + e == p1 - p2
    const float r = __fadd_rn(sh, __fadd_rn(e, __fsub_rn(p1l, p2l)));
    const uint32_t u = __float_as_uint(r);
    const float big = fmaxf(fabsf(p1), fabsf(p2));
    const bool clear_of_midpoints = ((u & 0xFFFFu) - 0x7FFEu) > 4u;
    proven = clear_of_midpoints && fabsf(r) >= big * 0x1p-10f && big >= 0x1p-60f && big <= 0x1p100f;
    return static_cast<uint16_t>((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}

// Kept out of line: it is rare, and the callers unroll dozens of rotations.
__device__ __noinline__ inline uint16_t rope_diff_of_products_f64(float x1, float y1, float x2, float y2) {
    return f64_to_bf16_rne(__dsub_rn(__dmul_rn(static_cast<double>(x1), static_cast<double>(y1)),
                                     __dmul_rn(static_cast<double>(x2), static_cast<double>(y2))));
}

// ---- per-head RMSNorm of one feature -------------------------------------------------------------

// y = bf16(bf16(v * rr) * w) with both roundings to nearest even of the fp64 products (the per-head
// RMSNorm of one feature; rr = 1 / rms as fp64, w a bf16 weight).  The first product is evaluated in
// fp32 with its residual (rr split in two floats), which provably rounds like the fp64 product when the
// result is three fp32 ulps clear of every midpoint between bf16 values; otherwise fp64 decides.  The
// second product of two bf16 values is exact in fp32.
// The rare fp64 ways out of rmsnorm_feature, kept out of line so that the common path holds no fp64.
__device__ __noinline__ inline uint16_t bf16_of_product_f64(float a, double b) {
    return f64_to_bf16_rne(__dmul_rn(static_cast<double>(a), b));
}

__device__ __forceinline__ uint16_t rmsnorm_feature(uint16_t v16, double rr, float rr_hi, float rr_lo, float wf) {
    const float v = bf16_bits_to_float(v16);
    const float pr = __fmul_rn(v, rr_hi);
    const float pl = __fmaf_rn(v, rr_hi, -pr);                        // exact residual of the product
    const float r = __fadd_rn(pr, __fmaf_rn(v, rr_lo, pl));
    const uint32_t u = __float_as_uint(r);
    const float mag = fabsf(pr);
    uint16_t y1 = static_cast<uint16_t>((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
    if (!((((u & 0xFFFFu) - 0x7FFEu) > 4u) && mag >= 0x1p-60f && mag <= 0x1p100f))
        y1 = bf16_of_product_f64(v, rr);
    const float y1f = bf16_bits_to_float(y1);
    const float q = __fmul_rn(y1f, wf);
    const float qmag = fabsf(q);
    if (!(qmag >= 0x1p-100f && qmag <= 0x1p100f))                     // zero, tiny, huge or NaN: the plain way
        return bf16_of_product_f64(y1f, static_cast<double>(wf));
    const uint32_t uq = __float_as_uint(q);
    return static_cast<uint16_t>((uq + 0x7FFFu + ((uq >> 16) & 1u)) >> 16);
}

}  // namespace acdev
