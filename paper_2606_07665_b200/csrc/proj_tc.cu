// Projections for batched decode on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// Same products and epilogues as qkv_prelude.cu (QKV projection + RoPE + KV append; output projection
// + residual), for batches too large for the warp-MMA kernel's 32-row tiles: from a few dozen rows on
// the contraction y[b, n] = sum_k x[b, k] W[n, k] stops being a weight stream and becomes a thin GEMM,
// so the batch becomes the M dimension of a tcgen05.mma (up to 128 rows per CTA: W is streamed from
// HBM once per 128 rows) with the accumulator in tensor memory.
//
// What sets the pace is how fast one SM pulls its share of W out of DRAM through TMA (about 40 GB/s
// per SM, whatever the ring depth), so the feature tiles are chosen to put a CTA on nearly every SM:
//   QKV      48 features per CTA = 24 rotary pairs (W rows i..i+23 and i+d/2.. of one head).  A head
//            has 64 pairs (d = 128), so three tiles start at pairs 0, 24 and 48: 144 CTAs for 48 head
//            slots.  The third tile holds 16 pairs; the 8 pairs' worth of W rows past the head are
//            zero-filled by TMA and cost no traffic.
//   QKV with prelude variants (per-head norm, partial or interleaved rotary)
//            64 features per CTA = 32 pairs, disjoint tiles (two per head for d = 128, one for d = 64)
//            that form a thread-block cluster: the norm needs the sum of squares over the whole head,
//            and a partial half-split rotation needs partners from the sister tile, both through
//            distributed shared memory.  Clusters of three 1-CTA-per-SM tiles left SMs idle; clusters
//            of two pack.  The epilogue parks the rounded accumulators in the idle ring and runs the
//            norm and the rotation with one warp per batch row and one lane per pair.
//   o_proj   32 consecutive output features per CTA (128 CTAs for N = 4096).
// Per CTA:
//   warp 0   producer: per 128-wide K chunk one 3-D TMA load of the x tile [x_rows x 2 x 64] and one
//            5-D TMA load of the W tile, both as 128-byte-swizzled K-major blocks, into a ring that is
//            as deep as shared memory allows (256 contiguous bytes of every W row per load);
//   warp 1   allocates the TMEM columns; its lane 0 and lane 0 of the last warp issue the tcgen05.mma
//            (M128, K16, bf16 -> fp32, eight or sixteen per chunk) from shared-memory descriptors, the
//            first the even chunks into one accumulator, the second the odd chunks into another, then
//            tcgen05.commit to hand the stage back to the producer, and a final commit each to release
//            the epilogue, which adds the two accumulators;
//   the other warps are the epilogue, one warp per 32 batch rows and group of columns (thread = one
//            batch row; 8 rotary pairs or 16 output features): they compute addresses and fetch angles
//            or residuals while the main loop runs, then read the accumulator with tcgen05.ld, round
//            to bf16, rotate / add the residual, and store.
// Every wait is bounded; TMEM is released on every path.
#include <math.h>

#include "ac_device.cuh"
#include "ac_internal.h"

namespace ac {
namespace {

using namespace acdev;

enum { TC_EPI_QKV_ROPE_APPEND = 0, TC_EPI_RESIDUAL_ADD = 1, TC_EPI_QKV_ROPE_VARIANT = 2 };

constexpr int TC_M = 128;                       // rows of the MMA tile: batch rows per CTA, at most
constexpr int TC_MAX_STAGES = 12;
constexpr int TC_RING_BYTES = 220 * 1024;       // holds as many stages as fit
constexpr int TC_BAR_OFFSET = TC_RING_BYTES;
constexpr int TC_SMEM_TOTAL = TC_BAR_OFFSET + (2 * TC_MAX_STAGES + 1) * 8 + 16 + 1024;

template <int EPI>
struct TcTile {
    // features per CTA: 48 (QKV; three overlapping tiles per head put a CTA on nearly every SM), 32
    // (o_proj), 64 (QKV with prelude variants: two disjoint tiles per head, which pair up as clusters
    // of two without leaving SMs idle the way clusters of three 1-CTA-per-SM tiles did)
    static constexpr int N = EPI == TC_EPI_RESIDUAL_ADD ? 32 : (EPI == TC_EPI_QKV_ROPE_VARIANT ? 64 : 48);
    static constexpr int GROUPS = N / 16;                                     // epilogue warps per 32 rows
    static constexpr int THREADS = 64 + 128 * GROUPS + 32;       // the last warp holds the second MMA issuer
    static constexpr int MMA2_WARP = 2 + 4 * GROUPS;
    static constexpr int B_BLOCK = N * 128;          // one swizzled [N rows x 128 B] block of W
    static constexpr uint32_t ACC_COLS = EPI == TC_EPI_RESIDUAL_ADD ? 32 : 64;       // a power of two >= N
    static constexpr uint32_t TMEM_COLS = 2 * ACC_COLS;                              // two accumulators
};

// First rotary pair of QKV tile `blk` inside its head: 24-pair tiles at 0, 24 and 48 (64 pairs per
// head) or at 0 and 24 (32 pairs per head).  The last tile reaches past the head: TMA fills those W
// rows with zeros without reading anything, and the epilogue skips the column groups that hold them.
__host__ __device__ inline int qkv_tile_first_pair(int /*half_d*/, int blk) { return 24 * blk; }

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
    // prelude variants only (TC_EPI_QKV_ROPE_VARIANT)
    int rotary_dim, interleaved;
    const uint16_t* q_norm_w;
    const uint16_t* k_norm_w;
    float norm_eps;
};

// Where the variant epilogue keeps its working set, in the shared memory of the (by then idle) ring.
// A feature row is 66 values long so that 32 threads, one batch row each, hit 32 different banks.
struct VariantSmem {
    static constexpr int ROW = 66;                                    // bf16 values per parked row
    static constexpr int VALS = 0;                                    // [128][ROW] rounded features
    static constexpr int VALSN = VALS + TC_M * ROW * 2;               // [128][ROW] after the norm
    static constexpr int PSUM = VALSN + TC_M * ROW * 2;               // [4 column groups][128] sums of squares
    static constexpr int RSCALE = PSUM + 4 * TC_M * 8;                // [128] 1 / rms of the row
    static constexpr int ROW_DST = RSCALE + TC_M * 8;                 // [128] destination rows
    static constexpr int ROW_CTX = ROW_DST + TC_M * 8;                // [128] position; -1: row not stored
    static constexpr int END = ROW_CTX + TC_M * 4;
    static_assert(PSUM % 8 == 0 && END <= TC_RING_BYTES, "variant epilogue working set");
};

// The variant epilogue's tiles are disjoint blocks of 32 pairs: tile blk holds pairs [32 blk, 32 blk + 32).
constexpr int kVariantTilePairs = 32;

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

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n (a multiple of 16).
__device__ __forceinline__ uint32_t umma_idesc_bf16_m128(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | ((128u >> 4) << 24);
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

// 32 lanes x 8 consecutive 32-bit columns: thread i of the warp gets lane (warp % 4) * 32 + i.
__device__ __forceinline__ void tmem_ld_32x8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// KBLK = 64-element (128-byte) K blocks per stage, 2 or 4 (a compile-time constant: the thread that
// issues the MMAs is the critical path of the main loop, and every instruction in its loop shows).
template <int EPI, int KBLK>
__global__ void __launch_bounds__(TcTile<EPI>::THREADS, 1) proj_tc_kernel(const __grid_constant__ CUtensorMap w_map,
                                                                          const __grid_constant__ CUtensorMap x_map,
                                                                          const TcParams p) {
    using T = TcTile<EPI>;
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

    const int blk = blockIdx.x;          // pair tile inside the head (QKV) / unused (o_proj)
    const int hh = blockIdx.y;           // head slot (QKV) / block of 32 output features (o_proj)
    const int pair0 = EPI == TC_EPI_RESIDUAL_ADD ? 0
                      : EPI == TC_EPI_QKV_ROPE_VARIANT ? kVariantTilePairs * blk : qkv_tile_first_pair(p.d / 2, blk);
    // The x box holds x_rows rows per 64-element block; the MMA always reads 128.  Rows past x_rows are
    // whatever the ring holds: every accumulator row depends on its own x row only, and the epilogue
    // skips them.  A stage is the x tile followed by the W tile.
    const int b0 = blockIdx.z * p.x_rows;
    const uint32_t a_block = static_cast<uint32_t>(p.x_rows) * 128u;
    const uint32_t a_bytes = KBLK * a_block;
    const uint32_t stage_bytes = a_bytes + KBLK * T::B_BLOCK;        // a multiple of 1024
    const int stages = min(TC_MAX_STAGES, TC_RING_BYTES / static_cast<int>(stage_bytes));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int n_chunks = (p.K + 64 * KBLK - 1) / (64 * KBLK);

    if (threadIdx.x == 0) {
        tma_prefetch_descriptor(&w_map);
        tma_prefetch_descriptor(&x_map);
        for (int s = 0; s < TC_MAX_STAGES; ++s) {
            mbar_init(full_bar + s * 8, 1);
            mbar_init(empty_bar + s * 8, 1);
        }
        mbar_init(done_bar, 2);                              // one arrival per MMA-issuing thread
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(tmem_slot, T::TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_d = *tmem_slot_gen;
    // Prelude variants.  After the accumulators are parked in shared memory, the norm and the rotation
    // run with one epilogue warp per batch row and one lane per rotary pair of the tile (both halves).
    // What does not depend on the accumulators is fetched under the main loop: this lane's two norm
    // weights here, the rotation geometry of its two features -- partner, table entry, which half; the
    // same for every row -- and, in the epilogue warps, the table entries of the warp's rows.
    constexpr int VWARPS = 4 * T::GROUPS;                    // epilogue warps
    constexpr int VROWS = (TC_M + VWARPS - 1) / VWARPS;      // rows per epilogue warp in those passes
    const int n_rows = max(0, min(p.x_rows, p.B - b0));      // batch rows this CTA holds
    uint16_t norm_w_lo = 0, norm_w_hi = 0;
    int v_feat[2] = {0, 0}, v_ri[2] = {0, 0}, v_pcol[2] = {0, 0}, v_owner[2] = {0, 0};
    bool v_rot[2] = {false, false}, v_first[2] = {false, false};
    float v_cs[VROWS][2], v_sn[VROWS][2];
    if (EPI == TC_EPI_QKV_ROPE_VARIANT) {
        const bool rotated_head = hh < p.Hq + p.Hkv;
        const uint16_t* nw = hh < p.Hq ? p.q_norm_w : (rotated_head ? p.k_norm_w : nullptr);
        const int half_d = p.d / 2, R = p.rotary_dim, half_r = R / 2;
        if (nw != nullptr) {
            norm_w_lo = nw[pair0 + lane];
            norm_w_hi = nw[half_d + pair0 + lane];
        }
#pragma unroll
        for (int hsel = 0; hsel < 2; ++hsel) {
            const int f = (hsel == 0 ? 0 : half_d) + pair0 + lane;           // feature inside the head
            v_feat[hsel] = f;
            v_rot[hsel] = rotated_head && f < R;
            int partner;
            if (p.interleaved) {
                v_ri[hsel] = f >> 1;
                v_first[hsel] = (f & 1) == 0;
                partner = v_first[hsel] ? f + 1 : f - 1;
            } else {
                v_first[hsel] = f < half_r;
                v_ri[hsel] = v_first[hsel] ? f : f - half_r;
                partner = v_first[hsel] ? f + half_r : f - half_r;
            }
            if (!v_rot[hsel]) partner = f;
            const int ppair = partner & (half_d - 1);                        // head_dim / 2 is 32 or 64
            v_owner[hsel] = ppair / kVariantTilePairs;
            v_pcol[hsel] = (partner >= half_d ? T::N / 2 : 0) + (ppair - kVariantTilePairs * v_owner[hsel]);
        }
#pragma unroll
        for (int it = 0; it < VROWS; ++it)
#pragma unroll
            for (int hsel = 0; hsel < 2; ++hsel) {
                v_cs[it][hsel] = 1.0f;
                v_sn[it][hsel] = 0.0f;
            }
    }
    // W does not come from the kernel before this one, x does: the producer sends the weight loads of
    // the first ring fill on their way before anybody waits for that kernel (with programmatic stream
    // serialization this CTA may be resident while the predecessor still runs).
    const int first_fill = n_chunks < stages ? n_chunks : stages;
    if (threadIdx.x == 0) {
        const uint64_t stream_once = l2_policy_evict_first();
        for (int c = 0; c < first_fill; ++c) {
            mbar_arrive_expect_tx(full_bar + c * 8, stage_bytes);
            tma_load_5d(smem_base + c * stage_bytes + a_bytes, &w_map, full_bar + c * 8, 0, pair0, 0, hh, c * KBLK,
                        stream_once);
        }
    }
    cudaGridDependencySynchronize();      // x (and the residual) come from the preceding kernel

    bool timed_out = false;
    if (warp == 0) {
        if (lane == 0) {
            const uint64_t stream_once = l2_policy_evict_first();
            const uint64_t keep = l2_policy_evict_last();
            for (int c = 0; c < first_fill; ++c)             // the x tiles of the first ring fill
                tma_load_3d(smem_base + c * stage_bytes, &x_map, full_bar + c * 8, 0, b0, c * KBLK, keep);
            int stage = first_fill == stages ? 0 : first_fill;
            uint32_t round = first_fill == stages ? 1 : 0;   // how often the ring has wrapped
            for (int c = first_fill; c < n_chunks; ++c) {
                if (round > 0 && !mbar_wait_bounded(empty_bar + stage * 8, (round - 1) & 1)) {
                    timed_out = true;
                    break;
                }
                const uint32_t dst = smem_base + stage * stage_bytes;
                mbar_arrive_expect_tx(full_bar + stage * 8, stage_bytes);
                tma_load_3d(dst, &x_map, full_bar + stage * 8, 0, b0, c * KBLK, keep);
                tma_load_5d(dst + a_bytes, &w_map, full_bar + stage * 8, 0, pair0, 0, hh, c * KBLK, stream_once);
                if (++stage == stages) {
                    stage = 0;
                    ++round;
                }
            }
        }
    } else if (warp == 1 || warp == T::MMA2_WARP) {
        // Two threads issue the MMAs, one the even chunks into the first accumulator, one the odd chunks
        // into the second (the epilogue adds them): a thread is held ~75 cycles per tcgen05.mma however
        // narrow the tile, several times the tensor pipe's own time here.  BOTH threads wait for EVERY
        // chunk's full barrier, in order: a thread that skipped the barriers of the other's chunks could
        // run a whole phase ahead of a stage, which a one-bit parity wait cannot tell from being on time.
        if (lane == 0) {
            const int which = warp == 1 ? 0 : 1;
            const uint32_t idesc = umma_idesc_bf16_m128(T::N);
            const uint32_t acc = tmem_d + which * T::ACC_COLS;
            int stage = 0;
            uint32_t round = 0;
            for (int c = 0; c < n_chunks; ++c) {
                if (!mbar_wait_bounded(full_bar + stage * 8, round & 1)) {
                    timed_out = true;
                    break;
                }
                if ((c & 1) == which) {
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_base + stage * stage_bytes;
#pragma unroll
                    for (int kb = 0; kb < KBLK; ++kb) {
                        const uint64_t adesc = umma_desc_k_major_sw128(a_addr + kb * a_block);
                        const uint64_t bdesc = umma_desc_k_major_sw128(a_addr + a_bytes + kb * T::B_BLOCK);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)       // 16 elements = 32 bytes = 2 descriptor units
                            umma_bf16(acc, adesc + 2 * ks, bdesc + 2 * ks, idesc, (c > 1 || kb > 0 || ks > 0) ? 1u : 0u);
                    }
                    umma_commit(empty_bar + stage * 8);      // the stage is free once these MMAs have read it
                }
                if (++stage == stages) {
                    stage = 0;
                    ++round;
                }
            }
            umma_commit(done_bar);                           // this thread's accumulator is complete (or as far as it got)
        }
    }
    if (timed_out && p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_WAIT_TIMEOUT);

    if (warp >= 2 && warp < T::MMA2_WARP) {
        // ---- epilogue: thread = batch row; warp = 32 rows x one group of columns --------------------
        // Everything that does not need the accumulator is done first, under the main loop.
        const int quarter = warp & 3;                        // TMEM lanes this warp may read
        const int group = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        const int b = b0 + row;
        bool ok = row < p.x_rows && b < p.B;
        const uint32_t lane_base = tmem_d + (static_cast<uint32_t>(quarter * 32) << 16);

        if (EPI == TC_EPI_RESIDUAL_ADD) {
            // 16 output features: columns 16 group .. 16 group + 15
            uint16_t* dst = nullptr;
            uint4 res[2] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
            if (ok) {
                const size_t idx = static_cast<size_t>(b) * p.N + T::N * hh + 16 * group;
                dst = p.residual_out + idx;
                res[0] = *reinterpret_cast<const uint4*>(p.residual_in + idx);
                res[1] = *reinterpret_cast<const uint4*>(p.residual_in + idx + 8);
            }
            const bool ready = mbar_wait_bounded(done_bar, 0);
            if (!ready && lane == 0 && p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_WAIT_TIMEOUT);
            tc_fence_after_sync();
            uint32_t acc[2][8], odd[2][8];
            tmem_ld_32x8(lane_base + 16 * group, acc[0]);
            tmem_ld_32x8(lane_base + 16 * group + 8, acc[1]);
            tmem_ld_32x8(lane_base + T::ACC_COLS + 16 * group, odd[0]);           // the odd chunks' sums
            tmem_ld_32x8(lane_base + T::ACC_COLS + 16 * group + 8, odd[1]);
            tmem_ld_wait();
            if (n_chunks > 1) {                              // a single chunk leaves the second accumulator unwritten
#pragma unroll
                for (int v = 0; v < 2; ++v)
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        acc[v][e] = __float_as_uint(__uint_as_float(acc[v][e]) + __uint_as_float(odd[v][e]));
            }
            if (ready && ok) {
#pragma unroll
                for (int v = 0; v < 2; ++v) {                // 8 features = 16 bytes at a time
                    const uint32_t rw[4] = {res[v].x, res[v].y, res[v].z, res[v].w};
                    uint32_t ow[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float r0 = __uint_as_float(rw[e] << 16);
                        const float r1 = __uint_as_float(rw[e] & 0xFFFF0000u);
                        ow[e] = pack_bf16x2(r0 + __uint_as_float(acc[v][2 * e]), r1 + __uint_as_float(acc[v][2 * e + 1]));
                    }
                    *reinterpret_cast<uint4*>(dst + v * 8) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                }
            }
        } else if (EPI == TC_EPI_QKV_ROPE_VARIANT) {
            // prelude variants: this warp only rounds its 8 pairs and parks them in shared memory (the
            // ring is free once the accumulators are complete); the norm and the rotation follow below,
            // by all threads of the CTA, because they reach across columns and across sister CTAs.
            // where the row goes (as in the plain epilogue), looked up under the main loop
            int ctx = -1;
            unsigned long long dst = 0;
            {
                // table entries of the rows this warp rotates later (rows warp - 2, + 16, ...); a full
                // half-split rotation turns both halves of a pair by the same entry
                const int half_r = p.rotary_dim / 2;
                const bool one_entry = v_rot[0] == v_rot[1] && v_ri[0] == v_ri[1];
#pragma unroll
                for (int it = 0; it < VROWS; ++it) {
                    const int prow = (warp - 2) + it * VWARPS;
                    if (prow >= n_rows) continue;            // the same for the whole warp
                    const int c = p.context_lens[b0 + prow];
                    const bool valid = c >= 0 && c < p.max_position;
                    // loads without a condition (entry 0 when there is nothing to rotate)
                    const size_t e0 = (valid && v_rot[0]) ? static_cast<size_t>(c) * half_r + v_ri[0] : 0;
                    v_cs[it][0] = __ldg(p.rope_cos + e0);
                    v_sn[it][0] = __ldg(p.rope_sin + e0);
                    if (one_entry) {
                        v_cs[it][1] = v_cs[it][0];
                        v_sn[it][1] = v_sn[it][0];
                    } else {
                        const size_t e1 = (valid && v_rot[1]) ? static_cast<size_t>(c) * half_r + v_ri[1] : 0;
                        v_cs[it][1] = __ldg(p.rope_cos + e1);
                        v_sn[it][1] = __ldg(p.rope_sin + e1);
                    }
                }
            }
            if (group == 0 && ok) {
                const bool is_q = hh < p.Hq, is_k = !is_q && hh < p.Hq + p.Hkv;
                ctx = p.context_lens[b];
                if (ctx >= 0) {
                    const int page_idx = ctx / p.page_size;
                    if (ctx >= p.max_position || page_idx >= p.max_pages_per_seq) {
                        if (p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_POSITION_OOB);
                        ctx = -1;
                    } else if (is_q) {
                        dst = reinterpret_cast<unsigned long long>(p.q_out + (static_cast<size_t>(b) * p.Hq + hh) * p.d);
                    } else {
                        const int page = p.block_table[static_cast<size_t>(b) * p.max_pages_per_seq + page_idx];
                        if (page < 0 || page >= p.num_pages) {
                            if (p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_PAGE_OOB);
                            ctx = -1;
                        } else {
                            const int h = is_k ? hh - p.Hq : hh - p.Hq - p.Hkv;
                            dst = reinterpret_cast<unsigned long long>(
                                (is_k ? p.k_cache : p.v_cache) + static_cast<size_t>(page) * p.stride_page +
                                static_cast<size_t>(ctx - page_idx * p.page_size) * p.stride_token +
                                static_cast<size_t>(h) * p.stride_head);
                        }
                    }
                }
            }
            const bool ready = mbar_wait_bounded(done_bar, 0);
            if (!ready && lane == 0 && p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_WAIT_TIMEOUT);
            tc_fence_after_sync();
            uint32_t lo[8], hi[8], lo_odd[8], hi_odd[8];
            tmem_ld_32x8(lane_base + 8 * group, lo);
            tmem_ld_32x8(lane_base + T::N / 2 + 8 * group, hi);
            tmem_ld_32x8(lane_base + T::ACC_COLS + 8 * group, lo_odd);
            tmem_ld_32x8(lane_base + T::ACC_COLS + T::N / 2 + 8 * group, hi_odd);
            tmem_ld_wait();
            uint32_t* vrow = reinterpret_cast<uint32_t*>(smem_gen + VariantSmem::VALS) + row * (VariantSmem::ROW / 2);
            double ss = 0.0;
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
                uint32_t pk[2];
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    float a = __uint_as_float(lo[e + t]), bq = __uint_as_float(hi[e + t]);
                    if (n_chunks > 1) {
                        a += __uint_as_float(lo_odd[e + t]);
                        bq += __uint_as_float(hi_odd[e + t]);
                    }
                    pk[t] = (ready && ok) ? pack_bf16x2(a, bq) : 0u;
                    const double ar = static_cast<double>(__uint_as_float(pk[t] << 16));
                    const double br = static_cast<double>(__uint_as_float(pk[t] & 0xFFFF0000u));
                    ss = __dadd_rn(ss, __dadd_rn(__dmul_rn(ar, ar), __dmul_rn(br, br)));
                }
                vrow[(8 * group + e) >> 1] = (pk[0] & 0xFFFFu) | (pk[1] << 16);
                vrow[(T::N / 2 + 8 * group + e) >> 1] = (pk[0] >> 16) | (pk[1] & 0xFFFF0000u);
            }
            reinterpret_cast<double*>(smem_gen + VariantSmem::PSUM)[group * TC_M + row] = ss;
            if (group == 0) {                                // the ring is free: these arrays live in it too
                reinterpret_cast<int*>(smem_gen + VariantSmem::ROW_CTX)[row] = ready ? ctx : -1;
                reinterpret_cast<unsigned long long*>(smem_gen + VariantSmem::ROW_DST)[row] = dst;
            }
        } else {
            // 8 rotary pairs: first halves in columns 8 group .., second halves in columns 24 + 8 group ..
            const int d = p.d, half_d = d / 2;
            const int i0 = pair0 + 8 * group;                // first pair of this warp inside the head
            ok = ok && i0 < half_d;                          // the last tile's columns past the head
            uint16_t* dst = nullptr;
            const bool rotate = hh < p.Hq + p.Hkv;           // v heads are stored as they are
            float cs[8], sn[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                cs[e] = 1.0f;
                sn[e] = 0.0f;
            }
            if (ok) {
                const int ctx = p.context_lens[b];
                int page_idx = 0;
                ok = ctx >= 0;
                if (ok) {
                    page_idx = ctx / p.page_size;
                    if (ctx >= p.max_position || page_idx >= p.max_pages_per_seq) {
                        if (p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_POSITION_OOB);
                        ok = false;
                    }
                }
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
                    const float* cos_row = p.rope_cos + static_cast<size_t>(ctx) * half_d + i0;
                    const float* sin_row = p.rope_sin + static_cast<size_t>(ctx) * half_d + i0;
                    const float4 ca = *reinterpret_cast<const float4*>(cos_row);
                    const float4 cb = *reinterpret_cast<const float4*>(cos_row + 4);
                    const float4 sa = *reinterpret_cast<const float4*>(sin_row);
                    const float4 sb = *reinterpret_cast<const float4*>(sin_row + 4);
                    cs[0] = ca.x; cs[1] = ca.y; cs[2] = ca.z; cs[3] = ca.w;
                    cs[4] = cb.x; cs[5] = cb.y; cs[6] = cb.z; cs[7] = cb.w;
                    sn[0] = sa.x; sn[1] = sa.y; sn[2] = sa.z; sn[3] = sa.w;
                    sn[4] = sb.x; sn[5] = sb.y; sn[6] = sb.z; sn[7] = sb.w;
                }
            }
            const bool ready = mbar_wait_bounded(done_bar, 0);
            if (!ready && lane == 0 && p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_WAIT_TIMEOUT);
            tc_fence_after_sync();
            uint32_t lo[8], hi[8], lo_odd[8], hi_odd[8];
            tmem_ld_32x8(lane_base + 8 * group, lo);                 // first halves of pairs i0 .. i0 + 7
            tmem_ld_32x8(lane_base + T::N / 2 + 8 * group, hi);      // their second halves
            tmem_ld_32x8(lane_base + T::ACC_COLS + 8 * group, lo_odd);                // the odd chunks' sums
            tmem_ld_32x8(lane_base + T::ACC_COLS + T::N / 2 + 8 * group, hi_odd);
            tmem_ld_wait();
            if (n_chunks > 1) {                              // a single chunk leaves the second accumulator unwritten
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    lo[e] = __float_as_uint(__uint_as_float(lo[e]) + __uint_as_float(lo_odd[e]));
                    hi[e] = __float_as_uint(__uint_as_float(hi[e]) + __uint_as_float(hi_odd[e]));
                }
            }
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
                        lo8[e] = rope_diff_of_products_f32(af[e], cs[e], bf[e], sn[e], p_lo);
                        hi8[e] = rope_diff_of_products_f32(bf[e], cs[e], af[e], -sn[e], p_hi);
                        unproven |= (p_lo ? 0u : 1u << e) | (p_hi ? 0u : 256u << e);
                    }
                    if (unproven != 0) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            if (unproven & (1u << e)) lo8[e] = rope_diff_of_products_f64(af[e], cs[e], bf[e], sn[e]);
                            if (unproven & (256u << e)) hi8[e] = rope_diff_of_products_f64(bf[e], cs[e], af[e], -sn[e]);
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
                *reinterpret_cast<uint4*>(dst + i0) = lo_v;
                *reinterpret_cast<uint4*>(dst + i0 + half_d) = hi_v;
            }
        }
    }
    if (EPI == TC_EPI_QKV_ROPE_VARIANT) {
        // ---- prelude variants: norm and rotation across the tiles of a head ----------------------------
        // The tiles of a head slot (blockIdx.x: two blocks of 32 pairs for head_dim 128, one for 64) are
        // one thread-block cluster.  With remote rotation partners three cluster barriers: parked features
        // and partial sums visible; normalised features visible; nobody's shared memory released while a
        // sister still reads it.  With local partners the sums are the only remote reads: one barrier
        // before them, and one whose arrival follows them and whose wait is the last thing the CTA does.
        // Every thread of every CTA of a cluster takes the same path through them.
        const int d = p.d;
        constexpr int VS = VariantSmem::ROW;
        uint16_t* vals = reinterpret_cast<uint16_t*>(smem_gen + VariantSmem::VALS);
        uint16_t* valsn = reinterpret_cast<uint16_t*>(smem_gen + VariantSmem::VALSN);
        double* psum = reinterpret_cast<double*>(smem_gen + VariantSmem::PSUM);
        double* rscale = reinterpret_cast<double*>(smem_gen + VariantSmem::RSCALE);
        int* row_ctx = reinterpret_cast<int*>(smem_gen + VariantSmem::ROW_CTX);
        unsigned long long* row_dst = reinterpret_cast<unsigned long long*>(smem_gen + VariantSmem::ROW_DST);
        const bool is_q = hh < p.Hq, is_k = !is_q && hh < p.Hq + p.Hkv;
        const uint16_t* norm_w = is_q ? p.q_norm_w : (is_k ? p.k_norm_w : nullptr);
        const int n_tiles = gridDim.x;
        const bool pass_warp = warp >= 2 && warp < T::MMA2_WARP;     // the epilogue warps run the passes
        static_assert(EPI != TC_EPI_QKV_ROPE_VARIANT || T::N / 2 == 32, "one lane per rotary pair of the tile");
        // A rotation partner sits in a sister's tile only for a half-split rotation over part of the head.
        // Both conditions are the same in every CTA of the cluster (same head slot, same parameters).
        const bool remote_partner = (is_q || is_k) && !p.interleaved && p.rotary_dim != d;
        const bool has_norm = norm_w != nullptr;
        if (has_norm || remote_partner) cluster_sync_all();   // everybody's parked features and partial sums
        else __syncthreads();
        if (norm_w != nullptr && threadIdx.x < n_rows) {
            double total = 0.0;
            for (int c = 0; c < n_tiles; ++c)
#pragma unroll
                for (int g = 0; g < T::GROUPS; ++g)
                    total = __dadd_rn(total, cluster_load_f64(cluster_map_shared(smem_addr(psum + g * TC_M + threadIdx.x), c)));
            // head_dim is a power of two: the mean is an exact scaling; 1 / x by the correctly rounded reciprocal
            rscale[threadIdx.x] = __drcp_rn(__dsqrt_rn(__dadd_rn(__dmul_rn(total, 1.0 / static_cast<double>(d)),
                                                                 static_cast<double>(p.norm_eps))));
        }
        __syncthreads();
        // Sisters read this CTA's partial sums above: it must not exit before they have.  With local
        // partners that is the last remote access, so arrive now and wait at the very end.
        const bool split_barrier = has_norm && !remote_partner;
        if (split_barrier) cluster_arrive_relaxed_all();      // publishes nothing: no release needed
        // Every sister of the cluster has the same head slot, hence the same answer to "is there a norm":
        // without one the rotation reads the parked features where they are.
        const uint16_t* rot_src = norm_w != nullptr ? valsn : vals;
        if (norm_w != nullptr && pass_warp) {
            const float w_lo = bf16_bits_to_float(norm_w_lo), w_hi = bf16_bits_to_float(norm_w_hi);
#pragma unroll
            for (int it = 0; it < VROWS; ++it) {
                const int row = (warp - 2) + it * VWARPS;
                if (row >= n_rows) continue;
                const double rr = rscale[row];
                const float rr_hi = __double2float_rn(rr);
                const float rr_lo = __double2float_rn(__dsub_rn(rr, static_cast<double>(rr_hi)));
#pragma unroll
                for (int hsel = 0; hsel < 2; ++hsel) {
                    const int item = row * VS + hsel * (T::N / 2) + lane;
                    valsn[item] = rmsnorm_feature(vals[item], rr, rr_hi, rr_lo, hsel == 0 ? w_lo : w_hi);
                }
            }
        }
        if (remote_partner) cluster_sync_all();               // the sisters' normalised features
        else __syncthreads();
        if (pass_warp) {
#pragma unroll
            for (int it = 0; it < VROWS; ++it) {
                const int row = (warp - 2) + it * VWARPS;
                if (row >= n_rows || row_ctx[row] < 0) continue;     // the same for the whole warp
                uint16_t* dst_row = reinterpret_cast<uint16_t*>(row_dst[row]);
#pragma unroll
                for (int hsel = 0; hsel < 2; ++hsel) {
                    uint16_t v16 = rot_src[row * VS + hsel * (T::N / 2) + lane];
                    if (v_rot[hsel]) {
                        const uint16_t* psrc = rot_src + row * VS + v_pcol[hsel];
                        const uint16_t other = v_owner[hsel] == blk
                                                   ? *psrc
                                                   : cluster_load_u16(cluster_map_shared(smem_addr(psrc), v_owner[hsel]));
                        // first half: x c - partner s; second half: x c + partner s
                        const float mine = bf16_bits_to_float(v16), theirs = bf16_bits_to_float(other);
                        const float s_signed = v_first[hsel] ? v_sn[it][hsel] : -v_sn[it][hsel];
                        bool proven;
                        v16 = rope_diff_of_products_f32(mine, v_cs[it][hsel], theirs, s_signed, proven);
                        if (!proven) v16 = rope_diff_of_products_f64(mine, v_cs[it][hsel], theirs, s_signed);
                    }
                    dst_row[v_feat[hsel]] = v16;
                }
            }
        }
        if (remote_partner) {                                 // nobody's shared memory goes while a sister reads it;
            cluster_arrive_relaxed_all();                     // nothing is published, so no wait for the stores above
            cluster_wait_all();
        } else if (split_barrier) {
            cluster_wait_all();
        }
    }

    // ---- release TMEM (every path reaches this point) ----------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_d, T::TMEM_COLS);
    }
}

template <int EPI, int KBLK>
cudaError_t launch_tc_k(const CUtensorMap& w_map, const CUtensorMap& x_map, const TcParams& p, dim3 grid,
                        cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(TcTile<EPI>::THREADS);
    cfg.dynamicSmemBytes = TC_SMEM_TOTAL;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;     // prelude variants: the tiles of a head slot
    attr[1].val.clusterDim.x = grid.x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = EPI == TC_EPI_QKV_ROPE_VARIANT ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, proj_tc_kernel<EPI, KBLK>, w_map, x_map, p);
}

template <int EPI>
cudaError_t launch_tc(const CUtensorMap& w_map, const CUtensorMap& x_map, const TcParams& p, int kblk, dim3 grid,
                      cudaStream_t stream) {
    return kblk == 4 ? launch_tc_k<EPI, 4>(w_map, x_map, p, grid, stream)
                     : launch_tc_k<EPI, 2>(w_map, x_map, p, grid, stream);
}

}  // namespace

// Batch rows per CTA: the batch is cut into the fewest tiles of at most 128 rows, of equal size rounded
// up to the 8-row swizzle period, so that no tile loads rows that do not exist.
int proj_tc_batch_rows(int B) {
    const int tiles = (B + TC_M - 1) / TC_M;
    const int rows = ((B + tiles - 1) / tiles + 7) / 8 * 8;
    return rows < TC_M ? rows : TC_M;
}

// K blocks per stage: 256-wide stages (sixteen MMAs per barrier round trip, 512 contiguous bytes per
// weight row and load) are faster, but only while at least five of them fit beside the x tiles -- with
// two threads issuing MMAs two stages are being read at any time, and the rest must cover the loads.
int proj_tc_k_blocks(int B) { return proj_tc_batch_rows(B) <= 40 ? 4 : 2; }

cudaError_t proj_tc_set_attributes(int smem_optin) {
    if (TC_SMEM_TOTAL > smem_optin) return cudaErrorInvalidConfiguration;
    cudaError_t e = cudaFuncSetAttribute(proj_tc_kernel<TC_EPI_QKV_ROPE_APPEND, 2>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_TOTAL);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(proj_tc_kernel<TC_EPI_QKV_ROPE_APPEND, 4>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_TOTAL);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(proj_tc_kernel<TC_EPI_RESIDUAL_ADD, 2>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_TOTAL);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(proj_tc_kernel<TC_EPI_RESIDUAL_ADD, 4>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_TOTAL);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(proj_tc_kernel<TC_EPI_QKV_ROPE_VARIANT, 2>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_TOTAL);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(proj_tc_kernel<TC_EPI_QKV_ROPE_VARIANT, 4>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_TOTAL);
    return e;
}

cudaError_t launch_qkv_rope_kv_append_tc(const CUtensorMap& w_map, const CUtensorMap& x_map, void* q_out,
                                         void* k_cache, void* v_cache, int64_t stride_page,
                                         int64_t stride_token, int64_t stride_head,
                                         const int32_t* block_table, int max_pages_per_seq,
                                         const int32_t* context_lens, const float* rope_cos,
                                         const float* rope_sin, int max_position, int B, int K, int Hq,
                                         int Hkv, int d, int page_size, int num_pages,
                                         int32_t* status_flag, const RopeVariant* variant, cudaStream_t stream) {
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
    const dim3 grid(d == 128 ? 3 : 2, Hq + 2 * Hkv, (B + p.x_rows - 1) / p.x_rows);
    if (variant != nullptr) {
        const dim3 vgrid(d / 2 / kVariantTilePairs, Hq + 2 * Hkv, (B + p.x_rows - 1) / p.x_rows);
        p.rotary_dim = variant->rotary_dim;
        p.interleaved = variant->interleaved;
        p.q_norm_w = static_cast<const uint16_t*>(variant->q_norm_weight);
        p.k_norm_w = static_cast<const uint16_t*>(variant->k_norm_weight);
        p.norm_eps = variant->norm_eps;
        return launch_tc<TC_EPI_QKV_ROPE_VARIANT>(w_map, x_map, p, proj_tc_k_blocks(B), vgrid, stream);
    }
    return launch_tc<TC_EPI_QKV_ROPE_APPEND>(w_map, x_map, p, proj_tc_k_blocks(B), grid, stream);
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
    return launch_tc<TC_EPI_RESIDUAL_ADD>(w_map, x_map, p, proj_tc_k_blocks(B), dim3(1, N / 32, (B + p.x_rows - 1) / p.x_rows), stream);
}

}  // namespace ac
