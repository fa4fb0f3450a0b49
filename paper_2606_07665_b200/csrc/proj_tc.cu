// Projections for batched decode on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// Same products and epilogues as qkv_prelude.cu (QKV projection + RoPE + KV append; output projection
// + residual), for batches too large for the warp-MMA kernel's 32-row tiles: from a few dozen rows on
// the contraction y[b, n] = sum_k x[b, k] W[n, k] stops being a weight stream and becomes a thin GEMM
// whose operand traffic is dominated by re-reading x, so a 128-row batch tile per CTA (W streamed from
// HBM once per 128 rows) and the UMMA pipe pay.
//
// One CTA = 128 batch rows (M) x 64 output features (N: 32 rotary pairs, i.e. W rows i..i+31 and
// i+d/2..i+d/2+31 of one head, or 64 consecutive rows for the output projection) x all of K.
//   warp 0   producer: per 128-wide K chunk one 3-D TMA load of the x tile [128 rows x 2 x 64] (32 KB;
//            rows beyond B are zero-filled by the bounds check) and one 5-D TMA load of the W tile
//            [2 halves x 32 rows x 2 x 64] (16 KB), both as 128-byte-swizzled K-major blocks, into a
//            4-stage ring (256 contiguous bytes of every W row per load);
//   warp 1   allocates 64 TMEM columns, and its lane 0 issues eight tcgen05.mma (M128 N64 K16, bf16
//            -> fp32) per chunk from shared-memory descriptors, then tcgen05.commit to hand the stage
//            back to the producer, and a final commit to release the epilogue;
//   warps 2-5 read the accumulator with tcgen05.ld (thread = one batch row, 64 columns), round to
//            bf16, rotate / add the residual, and store.
// Every wait is bounded; TMEM is released on every path.
#include <math.h>

#include "ac_device.cuh"
#include "ac_internal.h"

namespace ac {
namespace {

using namespace acdev;

enum { TC_EPI_QKV_ROPE_APPEND = 0, TC_EPI_RESIDUAL_ADD = 1 };

constexpr int TC_THREADS = 192;
constexpr int TC_M = 128;                       // rows of the MMA tile: batch rows per CTA, at most
constexpr int TC_N = 64;                        // output features per CTA
constexpr int TC_KBLK = 2;                      // 64-element (128-byte) K blocks per stage
constexpr int TC_KC = 64 * TC_KBLK;             // K elements per stage
constexpr int TC_MAX_STAGES = 12;
constexpr int TC_RING_BYTES = 216 * 1024;       // holds as many stages as fit: 4 at 128 batch rows, 8 at 40
constexpr int TC_B_BLOCK = TC_N * 128;          // one swizzled [64 rows x 128 B] block of W: 8 KB
constexpr int TC_B_BYTES = TC_KBLK * TC_B_BLOCK;
constexpr int TC_BAR_OFFSET = TC_RING_BYTES;
constexpr int TC_SMEM_TOTAL = TC_BAR_OFFSET + (2 * TC_MAX_STAGES + 1) * 8 + 16 + 1024;
constexpr uint32_t TC_TMEM_COLS = 64;

struct TcParams {
    uint16_t* q_out;
    uint16_t* k_cache;
    uint16_t* v_cache;
    int64_t stride_page, stride_token, stride_head;
    const int32_t* block_table;
    const int32_t* context_lens;
    const float* rope_cos;
    const float* rope_sin;
    int32_t* status_flag;
    int max_pages_per_seq, max_position, num_pages, page_size;
    int B, K, Hq, Hkv, d;
    int x_rows;                   // batch rows a CTA loads and owns: a multiple of 8, at most TC_M
    const uint16_t* residual_in;
    uint16_t* residual_out;
    int N;
};

// ---- tcgen05 wrappers ---------------------------------------------------------------------------

__device__ __forceinline__ void tmem_alloc(uint32_t smem_result_addr, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result_addr),
                 "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

__device__ __forceinline__ void tc_fence_before_sync() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_after_sync() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major, 128-byte-swizzled tile: rows are 128 bytes, groups of
// eight rows are 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_k_major_sw128(uint32_t smem_byte_addr) {
    uint64_t desc = 0;
    desc |= static_cast<uint64_t>((smem_byte_addr >> 4) & 0x3FFFu);       // start address
    desc |= static_cast<uint64_t>(1) << 16;                                // leading byte offset (unused here)
    desc |= static_cast<uint64_t>(1024 >> 4) << 32;                        // stride byte offset: 8 rows
    desc |= static_cast<uint64_t>(1) << 46;                                // descriptor version
    desc |= static_cast<uint64_t>(2) << 61;                                // 128-byte swizzle
    return desc;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 64.
__device__ __forceinline__ uint32_t umma_idesc_bf16_m128_n64() {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((TC_N >> 3) << 17) | ((TC_M >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Arrives on the mbarrier when all tensor-core operations issued so far by this thread are done.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp gets lane (warp % 4) * 32 + i.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

// 32 lanes x 8 consecutive 32-bit columns.
__device__ __forceinline__ void tmem_ld_32x8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

template <int EPI>
__global__ void __launch_bounds__(TC_THREADS, 1) proj_tc_kernel(const __grid_constant__ CUtensorMap w_map,
                                                                const __grid_constant__ CUtensorMap x_map,
                                                                const TcParams p) {
    cudaTriggerProgrammaticLaunchCompletion();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_addr(smem_raw));
    const uint32_t full_bar = smem_base + TC_BAR_OFFSET;
    const uint32_t empty_bar = full_bar + TC_MAX_STAGES * 8;
    const uint32_t done_bar = empty_bar + TC_MAX_STAGES * 8;
    const uint32_t tmem_slot = done_bar + 8;                       // 4 bytes: TMEM base address
    volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + TC_BAR_OFFSET +
                                                                            (2 * TC_MAX_STAGES + 1) * 8);

    const int blk = blockIdx.x;          // block of 32 pairs inside the head (QKV) / unused (o_proj)
    const int hh = blockIdx.y;           // head slot (QKV) / block of 64 output features (o_proj)
    // The x box holds x_rows rows per 64-element block; the MMA always reads 128.  Rows past x_rows are
    // whatever the ring holds: every accumulator row depends on its own x row only, and the epilogue
    // skips them.  A stage is the x tile followed by the W tile.  The weights come from DRAM with
    // microseconds of latency, so the ring is as deep as shared memory allows.
    const int b0 = blockIdx.z * p.x_rows;
    const uint32_t a_block = static_cast<uint32_t>(p.x_rows) * 128u;
    const uint32_t a_bytes = TC_KBLK * a_block;
    const uint32_t stage_bytes = a_bytes + TC_B_BYTES;       // a multiple of 1024
    const int stages = min(TC_MAX_STAGES, TC_RING_BYTES / static_cast<int>(stage_bytes));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int n_chunks = (p.K + TC_KC - 1) / TC_KC;

    if (threadIdx.x == 0) {
        tma_prefetch_descriptor(&w_map);
        tma_prefetch_descriptor(&x_map);
        for (int s = 0; s < TC_MAX_STAGES; ++s) {
            mbar_init(full_bar + s * 8, 1);
            mbar_init(empty_bar + s * 8, 1);
        }
        mbar_init(done_bar, 1);
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(tmem_slot, TC_TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_d = *tmem_slot_gen;
    cudaGridDependencySynchronize();      // x (and the residual) come from the preceding kernel

    bool timed_out = false;
    if (warp == 0) {
        if (lane == 0) {
            const uint64_t stream_once = l2_policy_evict_first();
            const uint64_t keep = l2_policy_evict_last();
            int stage = 0;
            uint32_t round = 0;                              // how often the ring has wrapped
            for (int c = 0; c < n_chunks; ++c) {
                if (round > 0 && !mbar_wait_bounded(empty_bar + stage * 8, (round - 1) & 1)) {
                    timed_out = true;
                    break;
                }
                const uint32_t dst = smem_base + stage * stage_bytes;
                mbar_arrive_expect_tx(full_bar + stage * 8, stage_bytes);
                tma_load_3d(dst, &x_map, full_bar + stage * 8, 0, b0, c * TC_KBLK, keep);
                if (EPI == TC_EPI_QKV_ROPE_APPEND)
                    tma_load_5d(dst + a_bytes, &w_map, full_bar + stage * 8, 0, 32 * blk, 0, hh, c * TC_KBLK,
                                stream_once);
                else
                    tma_load_5d(dst + a_bytes, &w_map, full_bar + stage * 8, 0, 0, 0, hh, c * TC_KBLK,
                                stream_once);
                if (++stage == stages) {
                    stage = 0;
                    ++round;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16_m128_n64();
            int stage = 0;
            uint32_t round = 0;
            for (int c = 0; c < n_chunks; ++c) {
                if (!mbar_wait_bounded(full_bar + stage * 8, round & 1)) {
                    timed_out = true;
                    break;
                }
                tc_fence_after_sync();
                const uint32_t a_addr = smem_base + stage * stage_bytes;
#pragma unroll
                for (int kb = 0; kb < TC_KBLK; ++kb) {
                    const uint64_t adesc = umma_desc_k_major_sw128(a_addr + kb * a_block);
                    const uint64_t bdesc = umma_desc_k_major_sw128(a_addr + a_bytes + kb * TC_B_BLOCK);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)           // 16 elements = 32 bytes = 2 descriptor units
                        umma_bf16(tmem_d, adesc + 2 * ks, bdesc + 2 * ks, idesc,
                                  (c > 0 || kb > 0 || ks > 0) ? 1u : 0u);
                }
                umma_commit(empty_bar + stage * 8);          // the stage is free once these MMAs have read it
                if (++stage == stages) {
                    stage = 0;
                    ++round;
                }
            }
            umma_commit(done_bar);                           // accumulator complete (or as far as we got)
        }
    }
    if (timed_out && p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_WAIT_TIMEOUT);

    if (warp >= 2) {
        // ---- epilogue: thread = batch row, 64 accumulator columns -------------------------------------
        // Everything that does not need the accumulator is done first, under the main loop: the row's
        // position, its destination and (QKV) its rotary angles.
        const int quarter = warp & 3;                        // TMEM lanes this warp may read
        const int row = quarter * 32 + lane;
        const int b = b0 + row;
        bool ok = row < p.x_rows && b < p.B;
        uint16_t* dst = nullptr;
        const uint16_t* res = nullptr;
        bool rotate = false;
        const float* cos_row = nullptr;                      // angles of this row's 32 pairs (QKV, q and k heads)
        const float* sin_row = nullptr;
        float c_nxt[8], s_nxt[8];                            // angles of the next group of 8 pairs
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            c_nxt[e] = 1.0f;
            s_nxt[e] = 0.0f;
        }
        const int i0 = 32 * blk;                             // first pair of this CTA (QKV)
        if (EPI == TC_EPI_RESIDUAL_ADD) {
            if (ok) {
                const size_t idx = static_cast<size_t>(b) * p.N + 64 * hh;
                dst = p.residual_out + idx;
                res = p.residual_in + idx;
            }
        } else if (ok) {
            const int ctx = p.context_lens[b];
            const int d = p.d, half_d = d / 2;
            int page_idx = 0;
            ok = ctx >= 0;
            if (ok) {
                page_idx = ctx / p.page_size;
                if (ctx >= p.max_position || page_idx >= p.max_pages_per_seq) {
                    if (p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_POSITION_OOB);
                    ok = false;
                }
            }
            rotate = hh < p.Hq + p.Hkv;
            if (ok) {
                if (hh < p.Hq) {
                    dst = p.q_out + (static_cast<size_t>(b) * p.Hq + hh) * d;
                } else {
                    const int page = p.block_table[static_cast<size_t>(b) * p.max_pages_per_seq + page_idx];
                    if (page < 0 || page >= p.num_pages) {
                        if (p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_PAGE_OOB);
                        ok = false;
                    } else {
                        const bool is_k = hh < p.Hq + p.Hkv;
                        const int h = is_k ? hh - p.Hq : hh - p.Hq - p.Hkv;
                        dst = (is_k ? p.k_cache : p.v_cache) + static_cast<size_t>(page) * p.stride_page +
                              static_cast<size_t>(ctx - page_idx * p.page_size) * p.stride_token +
                              static_cast<size_t>(h) * p.stride_head;
                    }
                }
            }
            if (ok && rotate) {
                cos_row = p.rope_cos + static_cast<size_t>(ctx) * half_d + i0;
                sin_row = p.rope_sin + static_cast<size_t>(ctx) * half_d + i0;
                const float4 ca = *reinterpret_cast<const float4*>(cos_row), cb = *reinterpret_cast<const float4*>(cos_row + 4);
                const float4 sa = *reinterpret_cast<const float4*>(sin_row), sb = *reinterpret_cast<const float4*>(sin_row + 4);
                c_nxt[0] = ca.x; c_nxt[1] = ca.y; c_nxt[2] = ca.z; c_nxt[3] = ca.w;
                c_nxt[4] = cb.x; c_nxt[5] = cb.y; c_nxt[6] = cb.z; c_nxt[7] = cb.w;
                s_nxt[0] = sa.x; s_nxt[1] = sa.y; s_nxt[2] = sa.z; s_nxt[3] = sa.w;
                s_nxt[4] = sb.x; s_nxt[5] = sb.y; s_nxt[6] = sb.z; s_nxt[7] = sb.w;
            }
        }

        const bool ready = mbar_wait_bounded(done_bar, 0);
        if (!ready && lane == 0 && p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_WAIT_TIMEOUT);
        tc_fence_after_sync();
        const uint32_t lane_base = tmem_d + (static_cast<uint32_t>(quarter * 32) << 16);
        if (EPI == TC_EPI_RESIDUAL_ADD) {
            uint32_t lo_bits[32], hi_bits[32];
            tmem_ld_32x32(lane_base, lo_bits);               // columns 0-31
            tmem_ld_32x32(lane_base + 32, hi_bits);          // columns 32-63
            tmem_ld_wait();
            if (ready && ok) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const uint32_t* acc = half == 0 ? lo_bits : hi_bits;
#pragma unroll
                    for (int v = 0; v < 4; ++v) {            // 8 features = 16 bytes at a time
                        const uint4 r8 = *reinterpret_cast<const uint4*>(res + half * 32 + v * 8);
                        const uint32_t rw[4] = {r8.x, r8.y, r8.z, r8.w};
                        uint32_t ow[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float r0 = __uint_as_float(rw[e] << 16);
                            const float r1 = __uint_as_float(rw[e] & 0xFFFF0000u);
                            ow[e] = pack_bf16x2(r0 + __uint_as_float(acc[v * 8 + 2 * e]),
                                                r1 + __uint_as_float(acc[v * 8 + 2 * e + 1]));
                        }
                        *reinterpret_cast<uint4*>(dst + half * 32 + v * 8) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                    }
                }
            }
        } else {
            // Four groups of 8 pairs in a rolled loop (the rotation code is long; unrolled 32 times it
            // would not stay in the instruction cache); the next group's angles are fetched a group ahead.
            const int half_d = p.d / 2;
#pragma unroll 1
            for (int v = 0; v < 4; ++v) {
                uint32_t lo[8], hi[8];
                tmem_ld_32x8(lane_base + v * 8, lo);         // first halves of pairs 8 v .. 8 v + 7
                tmem_ld_32x8(lane_base + 32 + v * 8, hi);    // their second halves
                float c_cur[8], s_cur[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    c_cur[e] = c_nxt[e];
                    s_cur[e] = s_nxt[e];
                }
                if (cos_row != nullptr && v < 3) {
                    const float4 ca = *reinterpret_cast<const float4*>(cos_row + (v + 1) * 8);
                    const float4 cb = *reinterpret_cast<const float4*>(cos_row + (v + 1) * 8 + 4);
                    const float4 sa = *reinterpret_cast<const float4*>(sin_row + (v + 1) * 8);
                    const float4 sb = *reinterpret_cast<const float4*>(sin_row + (v + 1) * 8 + 4);
                    c_nxt[0] = ca.x; c_nxt[1] = ca.y; c_nxt[2] = ca.z; c_nxt[3] = ca.w;
                    c_nxt[4] = cb.x; c_nxt[5] = cb.y; c_nxt[6] = cb.z; c_nxt[7] = cb.w;
                    s_nxt[0] = sa.x; s_nxt[1] = sa.y; s_nxt[2] = sa.z; s_nxt[3] = sa.w;
                    s_nxt[4] = sb.x; s_nxt[5] = sb.y; s_nxt[6] = sb.z; s_nxt[7] = sb.w;
                }
                tmem_ld_wait();
                if (ready && ok) {
                    uint16_t lo8[8], hi8[8];
                    float af[8], bf[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const uint32_t pk = pack_bf16x2(__uint_as_float(lo[e]), __uint_as_float(hi[e]));
                        lo8[e] = static_cast<uint16_t>(pk & 0xFFFFu);
                        hi8[e] = static_cast<uint16_t>(pk >> 16);
                        af[e] = __uint_as_float(pk << 16);
                        bf[e] = __uint_as_float(pk & 0xFFFF0000u);
                    }
                    if (rotate) {
                        // all sixteen rotations without a branch, then the rare unproven ones again in fp64
                        uint32_t unproven = 0;
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            bool p_lo, p_hi;
                            lo8[e] = rope_diff_of_products_f32(af[e], c_cur[e], bf[e], s_cur[e], p_lo);
                            hi8[e] = rope_diff_of_products_f32(bf[e], c_cur[e], af[e], -s_cur[e], p_hi);
                            unproven |= (p_lo ? 0u : 1u << e) | (p_hi ? 0u : 256u << e);
                        }
                        if (unproven != 0) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                if (unproven & (1u << e))
                                    lo8[e] = rope_diff_of_products_f64(af[e], c_cur[e], bf[e], s_cur[e]);
                                if (unproven & (256u << e))
                                    hi8[e] = rope_diff_of_products_f64(bf[e], c_cur[e], af[e], -s_cur[e]);
                            }
                        }
                    }
                    uint4 lo_v, hi_v;
                    lo_v.x = lo8[0] | (static_cast<uint32_t>(lo8[1]) << 16);
                    lo_v.y = lo8[2] | (static_cast<uint32_t>(lo8[3]) << 16);
                    lo_v.z = lo8[4] | (static_cast<uint32_t>(lo8[5]) << 16);
                    lo_v.w = lo8[6] | (static_cast<uint32_t>(lo8[7]) << 16);
                    hi_v.x = hi8[0] | (static_cast<uint32_t>(hi8[1]) << 16);
                    hi_v.y = hi8[2] | (static_cast<uint32_t>(hi8[3]) << 16);
                    hi_v.z = hi8[4] | (static_cast<uint32_t>(hi8[5]) << 16);
                    hi_v.w = hi8[6] | (static_cast<uint32_t>(hi8[7]) << 16);
                    *reinterpret_cast<uint4*>(dst + i0 + v * 8) = lo_v;
                    *reinterpret_cast<uint4*>(dst + i0 + half_d + v * 8) = hi_v;
                }
            }
        }
    }
    // ---- release TMEM (every path reaches this point) ----------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_d, TC_TMEM_COLS);
    }
}

template <int EPI>
cudaError_t launch_tc(const CUtensorMap& w_map, const CUtensorMap& x_map, const TcParams& p, dim3 grid,
                      cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = TC_SMEM_TOTAL;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, proj_tc_kernel<EPI>, w_map, x_map, p);
}

}  // namespace

// Batch rows per CTA: the batch is cut into the fewest tiles of at most 128 rows, of equal size rounded
// up to the 8-row swizzle period, so that no tile loads rows that do not exist.
int proj_tc_batch_rows(int B) {
    const int tiles = (B + TC_M - 1) / TC_M;
    const int rows = ((B + tiles - 1) / tiles + 7) / 8 * 8;
    return rows < TC_M ? rows : TC_M;
}

cudaError_t proj_tc_set_attributes(int smem_optin) {
    if (TC_SMEM_TOTAL > smem_optin) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(proj_tc_kernel<TC_EPI_QKV_ROPE_APPEND>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_TOTAL);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(proj_tc_kernel<TC_EPI_RESIDUAL_ADD>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_TOTAL);
}

cudaError_t launch_qkv_rope_kv_append_tc(const CUtensorMap& w_map, const CUtensorMap& x_map, void* q_out,
                                         void* k_cache, void* v_cache, int64_t stride_page,
                                         int64_t stride_token, int64_t stride_head,
                                         const int32_t* block_table, int max_pages_per_seq,
                                         const int32_t* context_lens, const float* rope_cos,
                                         const float* rope_sin, int max_position, int B, int K, int Hq,
                                         int Hkv, int d, int page_size, int num_pages,
                                         int32_t* status_flag, cudaStream_t stream) {
    TcParams p = {};
    p.q_out = static_cast<uint16_t*>(q_out);
    p.k_cache = static_cast<uint16_t*>(k_cache);
    p.v_cache = static_cast<uint16_t*>(v_cache);
    p.stride_page = stride_page;
    p.stride_token = stride_token;
    p.stride_head = stride_head;
    p.block_table = block_table;
    p.context_lens = context_lens;
    p.rope_cos = rope_cos;
    p.rope_sin = rope_sin;
    p.status_flag = status_flag;
    p.max_pages_per_seq = max_pages_per_seq;
    p.max_position = max_position;
    p.num_pages = num_pages;
    p.page_size = page_size;
    p.B = B;
    p.K = K;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.d = d;
    p.x_rows = proj_tc_batch_rows(B);
    return launch_tc<TC_EPI_QKV_ROPE_APPEND>(w_map, x_map, p,
                                             dim3(d / 64, Hq + 2 * Hkv, (B + p.x_rows - 1) / p.x_rows), stream);
}

cudaError_t launch_oproj_residual_tc(const CUtensorMap& w_map, const CUtensorMap& x_map,
                                     const void* residual_in, void* residual_out, int B, int K, int N,
                                     cudaStream_t stream) {
    TcParams p = {};
    p.B = B;
    p.K = K;
    p.N = N;
    p.residual_in = static_cast<const uint16_t*>(residual_in);
    p.residual_out = static_cast<uint16_t*>(residual_out);
    p.x_rows = proj_tc_batch_rows(B);
    return launch_tc<TC_EPI_RESIDUAL_ADD>(w_map, x_map, p, dim3(1, N / 64, (B + p.x_rows - 1) / p.x_rows), stream);
}

}  // namespace ac
