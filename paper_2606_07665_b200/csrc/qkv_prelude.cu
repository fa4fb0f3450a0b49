// Attention-prelude fusion: QKV projection (weight-streaming thin GEMM) + RoPE + KV append.
//
// y[b, n] = sum_k x[b, k] * W[n, k]  (x [B,H] bf16, W [(Hq+2Hkv)*d, H] bf16 in [N,K] layout, fp32
// accumulation), rounded to bf16; q and k features are then rotated at position context_lens[b] with
// the same exact-then-round arithmetic as the stand-alone RoPE kernel, q goes to q_out, k and v to
// the request's cache slot.  Nothing but the final results touches global memory.
//
// The kernel is bound by streaming W once from HBM.  One CTA owns 16 rotary pairs of one head: W rows
// i .. i+15 and i+d/2 .. i+d/2+15 (32 rows), all of K, one tile of 8 or 16 batch rows (larger batches
// run on the tcgen05 kernels); the grid is (d/32, Hq+2Hkv, batch tiles) -- 192 CTAs for a 32/8-head,
// d=128 layer.  A producer warp issues, per
// 256-wide K chunk, ONE 5-D tensor-map load for the 32 x 256 weight tile (the two row blocks and the
// four 64-element K blocks are box dimensions, so the 16 KB land as eight swizzled [16 x 128 B]
// blocks) and one 3-D load for the x tile, into a ring of stages guarded by full/empty mbarriers.
// Eight consumer warps split each chunk's sixteen k-steps; A fragments (W) and B fragments (x) come
// from shared memory by ldmatrix, products run on the bf16 m16n8k16 MMA (any batch size costs the
// same weight traffic).  At the end the warps' partial sums are reduced through shared memory and
// the epilogue rounds, rotates and scatters.
//
// The same weight-streaming body also serves the output projection (kernel family (v)): there a CTA
// owns 16 consecutive output features and the epilogue adds the residual row and rounds once; the
// RMSNorm that follows needs all H features of a row and runs as a second, dependent launch.
#include <math.h>

#include "ac_device.cuh"
#include "ac_internal.h"

namespace ac {
namespace {

using namespace acdev;

enum { EPI_QKV_ROPE_APPEND = 0, EPI_RESIDUAL_ADD = 1, EPI_QKV_ROPE_VARIANT = 2 };

constexpr int QKV_WARPS = 8;                          // consumer warps; warp QKV_WARPS produces
constexpr int QKV_THREADS = (QKV_WARPS + 1) * 32;
constexpr int KC = 256;                               // K elements per stage
constexpr int KBLOCKS = KC / 64;                      // 128-byte column blocks per stage
constexpr int W_BLOCK_BYTES = 16 * 128;               // one swizzled [16 rows x 64 elements] block
// Row blocks of 16 weight rows per CTA: 2 for the QKV projection (the first and second halves of 16
// rotary pairs), 1 for the output projection (16 consecutive features; 256 CTAs for N = 4096, so that
// most SMs stream for two CTAs -- 128 CTAs of 32 features left 20 SMs idle and the rest at the rate
// of a single CTA).
__host__ __device__ constexpr int row_blocks(int epi) { return epi == EPI_RESIDUAL_ADD ? 1 : 2; }

template <int BT, int RB>
struct QkvSmem {
    static constexpr int W_STAGE_BYTES = KBLOCKS * RB * W_BLOCK_BYTES;   // [kblock][row block][row][64]
    static constexpr int X_BLOCK_BYTES = BT * 128;                 // [BT batch rows x 64 elements]
    static constexpr int X_STAGE_BYTES = KBLOCKS * X_BLOCK_BYTES;
    static constexpr int STAGE_BYTES = W_STAGE_BYTES + X_STAGE_BYTES;
    static constexpr int STAGES = RB == 1 ? (BT <= 8 ? 8 : 6) : (BT <= 8 ? 5 : 4);
    static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
    static constexpr int TOTAL = BAR_OFFSET + 2 * STAGES * 8 + 1024;
    static_assert(QKV_WARPS * 16 * RB * BT * 4 <= STAGES * STAGE_BYTES, "reduction buffer must fit");
    // prelude variants: behind the reduction buffer, the CTA's rounded features [32][BT] (bf16 bits), the
    // same after the norm, and one fp64 sum of squares per batch row
    static constexpr int VAR_OFFSET = QKV_WARPS * 16 * RB * BT * 4;
    static constexpr int VAR_BYTES = 2 * 32 * BT * 2 + BT * 8;
    static_assert(RB != 2 || VAR_OFFSET + VAR_BYTES <= STAGES * STAGE_BYTES, "variant buffers must fit");
};

struct QkvParams {
    uint16_t* q_out;              // [B, Hq, d] rotated
    uint16_t* k_cache;
    uint16_t* v_cache;
    int64_t stride_page, stride_token, stride_head;
    const int32_t* block_table;
    const int32_t* context_lens;
    const float* rope_cos;
    const float* rope_sin;
    int32_t* status_flag;
    int max_pages_per_seq, max_position, num_pages, page_size;
    int B, H, Hq, Hkv, d;           // H = contraction length K of the product
    // output projection only
    const uint16_t* residual_in;  // [B, N] bf16
    uint16_t* residual_out;       // [B, N] bf16 (may alias residual_in)
    int N;                        // output features
    // prelude variants only (EPI_QKV_ROPE_VARIANT)
    int rotary_dim, interleaved;
    const uint16_t* q_norm_w;
    const uint16_t* k_norm_w;
    float norm_eps;
};

template <int BT, int EPI>
__global__ void __launch_bounds__(QKV_THREADS, 2) qkv_rope_append_kernel(
    const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap x_map,
    const QkvParams p) {
    constexpr int RB = row_blocks(EPI);
    constexpr int TROWS = 16 * RB;                    // weight rows (output features) per CTA
    constexpr int W_STAGE_BYTES = QkvSmem<BT, RB>::W_STAGE_BYTES;
    using L = QkvSmem<BT, RB>;
    constexpr int STAGES = L::STAGES;
    constexpr int NT = BT / 8;                        // 8-wide batch tiles of the MMA

    cudaTriggerProgrammaticLaunchCompletion();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_addr(smem_raw));
    const uint32_t full_bar = smem_base + L::BAR_OFFSET;
    const uint32_t empty_bar = full_bar + STAGES * 8;

    const int blk = blockIdx.x;                       // block of 16 rotary pairs inside the head
    const int hh = blockIdx.y;                        // head slot: q heads, then k heads, then v heads
    const int b0 = blockIdx.z * BT;                   // first batch row of this tile
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int n_chunks = (p.H + KC - 1) / KC;

    if (threadIdx.x == 0) {
        tma_prefetch_descriptor(&w_map);
        tma_prefetch_descriptor(&x_map);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar + s * 8, 1);
            mbar_init(empty_bar + s * 8, QKV_WARPS);
        }
        mbar_init_fence();
    }
    __syncthreads();
    // x is produced by the kernel before this one; W is not.  The producer thread therefore sends the
    // weight loads of the first ring fill on their way BEFORE it waits for that kernel (launched with
    // programmatic stream serialization this CTA may be resident while the predecessor still runs),
    // and everybody else waits here.
    if (warp != QKV_WARPS) cudaGridDependencySynchronize();

    // Prelude variants: in the epilogue consumer thread t owns items t and t + 256 of the CTA's
    // [32 features][BT rows] tile.  Where an item goes, which table entry turns it and where its partner
    // sits do not depend on the accumulators: looked up here, the loads complete under the main loop.
    constexpr int VTHREADS = QKV_WARPS * 32;
    constexpr int VITEMS = (32 * BT + VTHREADS - 1) / VTHREADS;
    uint16_t* v_dst[VITEMS];                          // where the item is stored; nullptr: not stored
    float v_cos[VITEMS], v_sin[VITEMS], v_w[VITEMS];   // table entry; norm weight of the feature
    int v_prow[VITEMS], v_owner[VITEMS], v_feat[VITEMS];
    bool v_rot[VITEMS], v_first[VITEMS];
    if (EPI == EPI_QKV_ROPE_VARIANT && warp != QKV_WARPS) {
        const int d = p.d, half_d = d / 2, R = p.rotary_dim, half_r = R / 2;
        const bool is_q = hh < p.Hq, is_k = !is_q && hh < p.Hq + p.Hkv;
        const uint16_t* nw = is_q ? p.q_norm_w : (is_k ? p.k_norm_w : nullptr);
#pragma unroll
        for (int k = 0; k < VITEMS; ++k) {
            const int item = threadIdx.x + k * VTHREADS;
            const int r = (item / BT) & 31, n = item % BT;
            const int b = b0 + n;
            const int f = (r >> 4) * half_d + 16 * blk + (r & 15);               // feature inside the head
            v_feat[k] = f;
            v_w[k] = nw != nullptr ? bf16_bits_to_float(nw[f]) : 1.0f;
            v_dst[k] = nullptr;
            v_cos[k] = 1.0f;
            v_sin[k] = 0.0f;
            v_rot[k] = (is_q || is_k) && f < R;
            int i, partner;
            if (p.interleaved) {
                i = f >> 1;
                v_first[k] = (f & 1) == 0;
                partner = v_first[k] ? f + 1 : f - 1;
            } else {
                v_first[k] = f < half_r;
                i = v_first[k] ? f : f - half_r;
                partner = v_first[k] ? f + half_r : f - half_r;
            }
            if (!v_rot[k]) partner = f;
            // the partner feature lives in CTA (partner mod d/2) / 16 of the cluster, local row below
            v_owner[k] = (partner & (half_d - 1)) >> 4;                          // d/2 is 32 or 64
            v_prow[k] = (partner >= half_d ? 16 : 0) + (partner & 15);
            if (item >= 32 * BT || b >= p.B) continue;
            const int ctx = p.context_lens[b];
            if (ctx < 0) continue;                         // inactive row
            const int page_idx = ctx / p.page_size;
            if (ctx >= p.max_position || page_idx >= p.max_pages_per_seq) {
                if (p.status_flag != nullptr && r == 0 && blk == 0) atomicOr(p.status_flag, AC_FLAG_POSITION_OOB);
                continue;
            }
            if (is_q) {
                v_dst[k] = p.q_out + (static_cast<size_t>(b) * p.Hq + hh) * d + f;
            } else {
                const int page = p.block_table[static_cast<size_t>(b) * p.max_pages_per_seq + page_idx];
                if (page < 0 || page >= p.num_pages) {
                    if (p.status_flag != nullptr && r == 0 && blk == 0) atomicOr(p.status_flag, AC_FLAG_PAGE_OOB);
                    continue;
                }
                const int h = is_k ? hh - p.Hq : hh - p.Hq - p.Hkv;
                v_dst[k] = (is_k ? p.k_cache : p.v_cache) + static_cast<size_t>(page) * p.stride_page +
                           static_cast<size_t>(ctx - page_idx * p.page_size) * p.stride_token +
                           static_cast<size_t>(h) * p.stride_head + f;
            }
            if (v_rot[k]) {
                v_cos[k] = __ldg(p.rope_cos + static_cast<size_t>(ctx) * half_r + i);
                v_sin[k] = __ldg(p.rope_sin + static_cast<size_t>(ctx) * half_r + i);
            }
        }
    }

    // The plain epilogues likewise: consumer thread t owns item t of the CTA's tile (one rotary pair, or one
    // output feature, of one batch row).  Its position, destination and angle -- or its residual -- are
    // fetched here, under the main loop, not behind it.
    uint16_t* e_dst = nullptr;                        // QKV: the head vector the pair goes to; nullptr: not stored
    float e_cos = 1.0f, e_sin = 0.0f;
    float e_res = 0.0f;                               // o_proj: the residual
    size_t e_idx = 0;
    bool e_live = false;
    if (EPI == EPI_QKV_ROPE_APPEND && warp != QKV_WARPS && threadIdx.x < 16 * BT) {
        const int j = threadIdx.x / BT, n = threadIdx.x % BT;     // pair inside the block, batch row
        const int b = b0 + n;
        const int ctx = b < p.B ? p.context_lens[b] : -1;
        if (ctx >= 0) {                                            // else: no such row, or inactive
            const int d = p.d, i = 16 * blk + j;                   // pair index inside the head
            const int page_idx = ctx / p.page_size;
            if (ctx >= p.max_position || page_idx >= p.max_pages_per_seq) {
                if (p.status_flag != nullptr && j == 0 && blk == 0) atomicOr(p.status_flag, AC_FLAG_POSITION_OOB);
            } else if (hh < p.Hq) {
                e_dst = p.q_out + (static_cast<size_t>(b) * p.Hq + hh) * d + i;
            } else {
                const int page = p.block_table[static_cast<size_t>(b) * p.max_pages_per_seq + page_idx];
                if (page < 0 || page >= p.num_pages) {
                    if (p.status_flag != nullptr && j == 0 && blk == 0) atomicOr(p.status_flag, AC_FLAG_PAGE_OOB);
                } else {
                    const bool is_k = hh < p.Hq + p.Hkv;
                    const int h = is_k ? hh - p.Hq : hh - p.Hq - p.Hkv;
                    e_dst = (is_k ? p.k_cache : p.v_cache) + static_cast<size_t>(page) * p.stride_page +
                            static_cast<size_t>(ctx - page_idx * p.page_size) * p.stride_token +
                            static_cast<size_t>(h) * p.stride_head + i;
                }
            }
            if (e_dst != nullptr && hh < p.Hq + p.Hkv) {           // q and k features are rotated
                e_cos = __ldg(p.rope_cos + static_cast<size_t>(ctx) * (d / 2) + i);
                e_sin = __ldg(p.rope_sin + static_cast<size_t>(ctx) * (d / 2) + i);
            }
        }
    }
    if (EPI == EPI_RESIDUAL_ADD && warp != QKV_WARPS && threadIdx.x < TROWS * BT) {
        const int r = threadIdx.x / BT, n = threadIdx.x % BT;     // feature inside the CTA's block, batch row
        const int b = b0 + n;
        if (b < p.B) {
            e_live = true;
            e_idx = static_cast<size_t>(b) * p.N + TROWS * hh + r;
            e_res = bf16_bits_to_float(p.residual_in[e_idx]);
        }
    }

    bool timed_out = false;
    float acc[RB][NT][4];
#pragma unroll
    for (int rb = 0; rb < RB; ++rb)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[rb][nt][e] = 0.0f;

    if (warp == QKV_WARPS) {
        // ---- producer: one thread streams the K chunks through the ring ----------------------------
        if (lane == 0) {
            const uint64_t stream_once = l2_policy_evict_first();
            const uint64_t keep = l2_policy_evict_last();
            const int first_fill = n_chunks < STAGES ? n_chunks : STAGES;
            for (int c = 0; c < first_fill; ++c) {          // weights of the first ring fill
                mbar_arrive_expect_tx(full_bar + c * 8, L::STAGE_BYTES);
                tma_load_5d(smem_base + c * L::STAGE_BYTES, &w_map, full_bar + c * 8, 0, 16 * blk, 0, hh,
                            c * KBLOCKS, stream_once);
            }
            cudaGridDependencySynchronize();
            for (int c = 0; c < first_fill; ++c)             // their x tiles
                tma_load_3d(smem_base + c * L::STAGE_BYTES + W_STAGE_BYTES, &x_map, full_bar + c * 8, 0, b0,
                            c * KBLOCKS, keep);
            for (int c = first_fill; c < n_chunks; ++c) {
                const int stage = c % STAGES;
                if (!mbar_wait_bounded(empty_bar + stage * 8, ((c / STAGES) - 1) & 1)) {
                    timed_out = true;
                    break;
                }
                const uint32_t dst = smem_base + stage * L::STAGE_BYTES;
                mbar_arrive_expect_tx(full_bar + stage * 8, L::STAGE_BYTES);
                tma_load_5d(dst, &w_map, full_bar + stage * 8, 0, 16 * blk, 0, hh, c * KBLOCKS, stream_once);
                tma_load_3d(dst + W_STAGE_BYTES, &x_map, full_bar + stage * 8, 0, b0, c * KBLOCKS, keep);
            }
        } else {
            cudaGridDependencySynchronize();               // the producer warp's other lanes
        }
    } else {
        // ---- consumers: warp w takes k-steps 2w and 2w+1 of every chunk ------------------------------
        const int mi = lane >> 3, r8 = lane & 7;
        const uint32_t a_row_off = ((mi & 1) * 8 + r8) * 128;    // A: matrices 0,2 rows 0-7; 1,3 rows 8-15
        const int a_chunk = mi >> 1;                              //    matrices 0,1 k lo; 2,3 k hi
        const uint32_t b_row_off = ((mi >> 1) * 8 + r8) * 128;   // B: matrices 0,1 batch 0-7; 2,3 batch 8-15
        const int b_chunk = mi & 1;                               //    matrices 0,2 k lo; 1,3 k hi
        for (int c = 0; c < n_chunks; ++c) {
            const int stage = c % STAGES;
            if (!mbar_wait_bounded(full_bar + stage * 8, (c / STAGES) & 1)) {
                timed_out = true;
                break;
            }
            const uint32_t wbase = smem_base + stage * L::STAGE_BYTES;
            const uint32_t xbase = wbase + W_STAGE_BYTES;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int ks = 2 * warp + u;                      // k-step (16 elements) inside the chunk
                const int kb = ks >> 2;                           // 64-element block
                const int ch = (ks & 3) * 2;                      // first 16-byte chunk of the k-step
                uint32_t a[RB][4];
#pragma unroll
                for (int rb = 0; rb < RB; ++rb) {
                    const uint32_t addr = wbase + (kb * RB + rb) * W_BLOCK_BYTES + a_row_off +
                                          (((ch + a_chunk) ^ r8) << 4);
                    ldmatrix_x4(a[rb][0], a[rb][1], a[rb][2], a[rb][3], addr);
                }
                if (NT == 1) {
                    // eight batch rows: two 8x8 matrices (k lo, k hi); lanes 16-31 repeat valid addresses
                    const uint32_t addr = xbase + kb * L::X_BLOCK_BYTES + r8 * 128 + (((ch + b_chunk) ^ r8) << 4);
                    uint32_t bq0, bq1, bq2, bq3;
                    ldmatrix_x4(bq0, bq1, bq2, bq3, addr);
                    (void)bq2;
                    (void)bq3;
#pragma unroll
                    for (int rb = 0; rb < RB; ++rb)
                        mma_bf16_16816(acc[rb][0][0], acc[rb][0][1], acc[rb][0][2], acc[rb][0][3], a[rb][0],
                                       a[rb][1], a[rb][2], a[rb][3], bq0, bq1);
                } else {
#pragma unroll
                    for (int np = 0; np < NT / 2; ++np) {
                        const uint32_t addr = xbase + kb * L::X_BLOCK_BYTES + np * 16 * 128 + b_row_off +
                                              (((ch + b_chunk) ^ r8) << 4);
                        uint32_t bq0, bq1, bq2, bq3;
                        ldmatrix_x4(bq0, bq1, bq2, bq3, addr);
#pragma unroll
                        for (int rb = 0; rb < RB; ++rb) {
                            mma_bf16_16816(acc[rb][2 * np][0], acc[rb][2 * np][1], acc[rb][2 * np][2],
                                           acc[rb][2 * np][3], a[rb][0], a[rb][1], a[rb][2], a[rb][3], bq0, bq1);
                            mma_bf16_16816(acc[rb][2 * np + 1][0], acc[rb][2 * np + 1][1], acc[rb][2 * np + 1][2],
                                           acc[rb][2 * np + 1][3], a[rb][0], a[rb][1], a[rb][2], a[rb][3], bq2, bq3);
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar + stage * 8);
        }
    }
    if (timed_out && lane == 0 && p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_WAIT_TIMEOUT);

    // ---- reduce the warps' partial sums through shared memory ----------------------------------------
    __syncthreads();                                   // every load has landed and been consumed
    float* red = reinterpret_cast<float*>(smem_gen);   // [QKV_WARPS][TROWS][BT]
    if (warp < QKV_WARPS) {
        const int g = lane >> 2, t = lane & 3;
#pragma unroll
        for (int rb = 0; rb < RB; ++rb)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                float* base = red + (warp * TROWS + rb * 16) * BT + nt * 8 + 2 * t;
                *reinterpret_cast<float2*>(base + g * BT) = make_float2(acc[rb][nt][0], acc[rb][nt][1]);
                *reinterpret_cast<float2*>(base + (g + 8) * BT) = make_float2(acc[rb][nt][2], acc[rb][nt][3]);
            }
    }
    __syncthreads();

    if (EPI == EPI_RESIDUAL_ADD) {
        // ---- epilogue of the output projection: h = bf16(residual + y), one rounding ----------------
        static_assert(EPI != EPI_RESIDUAL_ADD || TROWS * 16 <= QKV_WARPS * 32, "one item per consumer thread");
        if (e_live) {
            const int r = threadIdx.x / BT, n = threadIdx.x % BT;
            float y = 0.0f;
#pragma unroll
            for (int w = 0; w < QKV_WARPS; ++w) y += red[(w * TROWS + r) * BT + n];
            p.residual_out[e_idx] = static_cast<uint16_t>(pack_bf16x2(e_res + y, 0.0f) & 0xFFFFu);
        }
        return;
    }

    if (EPI == EPI_QKV_ROPE_VARIANT) {
        // ---- epilogue with the prelude variants ------------------------------------------------------
        // The d/32 CTAs that share a head (blockIdx.x) are one thread-block cluster.  A CTA holds 32 of
        // the head's features; the per-head RMSNorm needs the sum of squares of all d, and a half-split
        // rotation over part of the head pairs a feature with one that lives in a sister CTA.  So: every
        // CTA parks its rounded features and their partial sums of squares in shared memory, a cluster
        // barrier publishes them, the norm reads the sister CTAs' sums (fp64, exact, fixed order) and
        // parks the normalised features, and the rotation fetches each partner from whichever CTA owns
        // it.  With remote partners two more cluster barriers follow (normalised features visible;
        // nobody's shared memory released while a sister reads it); with local partners the sums are the
        // only remote reads: the CTA arrives at a second barrier once it has read them and waits for it
        // as the last thing it does.  All CTAs of a cluster take the same path (same head, same parameters).
        const int d = p.d;
        uint16_t* vals = reinterpret_cast<uint16_t*>(smem_gen + L::VAR_OFFSET);      // [32][BT]
        uint16_t* valsn = vals + 32 * BT;                                            // [32][BT] after the norm
        double* sums = reinterpret_cast<double*>(valsn + 32 * BT);                   // [BT]
        const bool is_q = hh < p.Hq, is_k = !is_q && hh < p.Hq + p.Hkv;
        const uint16_t* norm_w = is_q ? p.q_norm_w : (is_k ? p.k_norm_w : nullptr);
        const bool has_norm = norm_w != nullptr;
        const bool remote_partner = (is_q || is_k) && !p.interleaved && p.rotary_dim != d;
        const int n_cta = d / 32;                       // CTAs in the cluster
        const bool pass_thread = warp != QKV_WARPS;     // the consumer threads own the items
        if (pass_thread) {
#pragma unroll
            for (int k = 0; k < VITEMS; ++k) {
                const int item = threadIdx.x + k * VTHREADS;
                if (item >= 32 * BT) continue;
                const int r = item / BT, n = item - r * BT;
                float y = 0.0f;
#pragma unroll
                for (int w = 0; w < QKV_WARPS; ++w) y += red[(w * TROWS + r) * BT + n];
                vals[item] = static_cast<uint16_t>(pack_bf16x2(y, 0.0f) & 0xFFFFu);
            }
        }
        __syncthreads();
        if (has_norm && threadIdx.x < BT) {
            double ss = 0.0;
            for (int r = 0; r < 32; ++r) {
                const double v = static_cast<double>(bf16_bits_to_float(vals[r * BT + threadIdx.x]));
                ss = __dadd_rn(ss, __dmul_rn(v, v));
            }
            sums[threadIdx.x] = ss;
        }
        if (has_norm || remote_partner) cluster_sync_all();
        else __syncthreads();
        __shared__ double s_rscale[16];                 // 1 / rms of each batch row of the tile
        if (has_norm && threadIdx.x < BT) {
            double total = 0.0;
            for (int c = 0; c < n_cta; ++c)
                total = __dadd_rn(total, cluster_load_f64(cluster_map_shared(smem_addr(sums + threadIdx.x), c)));
            // head_dim is a power of two: the mean is an exact scaling; 1 / x by the correctly rounded reciprocal
            s_rscale[threadIdx.x] = __drcp_rn(__dsqrt_rn(__dadd_rn(__dmul_rn(total, 1.0 / static_cast<double>(d)),
                                                                   static_cast<double>(p.norm_eps))));
        }
        __syncthreads();
        const bool split_barrier = has_norm && !remote_partner;
        if (split_barrier) cluster_arrive_relaxed_all();      // publishes nothing: no release needed
        const uint16_t* rot_src = has_norm ? valsn : vals;
        if (has_norm && pass_thread) {
#pragma unroll
            for (int k = 0; k < VITEMS; ++k) {
                const int item = threadIdx.x + k * VTHREADS;
                if (item >= 32 * BT) continue;
                const double rr = s_rscale[item % BT];
                const float rr_hi = __double2float_rn(rr);
                const float rr_lo = __double2float_rn(__dsub_rn(rr, static_cast<double>(rr_hi)));
                valsn[item] = rmsnorm_feature(vals[item], rr, rr_hi, rr_lo, v_w[k]);
            }
        }
        if (remote_partner) cluster_sync_all();
        else __syncthreads();
        if (pass_thread) {
#pragma unroll
            for (int k = 0; k < VITEMS; ++k) {
                const int item = threadIdx.x + k * VTHREADS;
                if (item >= 32 * BT || v_dst[k] == nullptr) continue;
                const int n = item % BT;
                uint16_t v16 = rot_src[item];
                if (v_rot[k]) {
                    const uint16_t* psrc = rot_src + v_prow[k] * BT + n;
                    const uint16_t other =
                        v_owner[k] == blk ? *psrc : cluster_load_u16(cluster_map_shared(smem_addr(psrc), v_owner[k]));
                    // first half: x c - partner s; second half: x c + partner s
                    const float mine = bf16_bits_to_float(v16), theirs = bf16_bits_to_float(other);
                    const float s_signed = v_first[k] ? v_sin[k] : -v_sin[k];
                    bool proven;
                    v16 = rope_diff_of_products_f32(mine, v_cos[k], theirs, s_signed, proven);
                    if (!proven) v16 = rope_diff_of_products_f64(mine, v_cos[k], theirs, s_signed);
                }
                *v_dst[k] = v16;
            }
        }
        if (remote_partner) {                           // nothing is published here: no wait for the stores above
            cluster_arrive_relaxed_all();
            cluster_wait_all();
        } else if (split_barrier) {
            cluster_wait_all();
        }
        return;
    }

    // ---- epilogue: round, rotate, scatter --------------------------------------------------------
    if (e_dst != nullptr) {
        const int j = threadIdx.x / BT, n = threadIdx.x % BT;
        float y_lo = 0.0f, y_hi = 0.0f;
#pragma unroll
        for (int w = 0; w < QKV_WARPS; ++w) {
            y_lo += red[(w * TROWS + j) * BT + n];
            y_hi += red[(w * TROWS + 16 + j) * BT + n];
        }
        const uint32_t packed = pack_bf16x2(y_lo, y_hi);
        uint16_t lo = static_cast<uint16_t>(packed & 0xFFFFu), hi = static_cast<uint16_t>(packed >> 16);
        if (hh < p.Hq + p.Hkv) {                       // q and k features are rotated
            const uint16_t r0 = rope_first_half(lo, hi, e_cos, e_sin);
            const uint16_t r1 = rope_second_half(lo, hi, e_cos, e_sin);
            lo = r0;
            hi = r1;
        }
        e_dst[0] = lo;
        e_dst[p.d / 2] = hi;
    }
}

template <int BT, int EPI>
cudaError_t launch_qkv(const CUtensorMap& w_map, const CUtensorMap& x_map, const QkvParams& p,
                       cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = EPI == EPI_RESIDUAL_ADD ? dim3(1, p.N / (16 * row_blocks(EPI)), (p.B + BT - 1) / BT)
                                          : dim3(p.d / 32, p.Hq + 2 * p.Hkv, (p.B + BT - 1) / BT);
    cfg.blockDim = dim3(QKV_THREADS);
    cfg.dynamicSmemBytes = QkvSmem<BT, row_blocks(EPI)>::TOTAL;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;     // prelude variants: the CTAs of a head
    attr[1].val.clusterDim.x = static_cast<unsigned>(p.d / 32);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = EPI == EPI_QKV_ROPE_VARIANT ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, qkv_rope_append_kernel<BT, EPI>, w_map, x_map, p);
}

}  // namespace

cudaError_t qkv_set_attributes(int smem_optin) {
    if (QkvSmem<16, 2>::TOTAL > smem_optin || QkvSmem<16, 1>::TOTAL > smem_optin)
        return cudaErrorInvalidConfiguration;
    cudaError_t e;
#define AC_SET(BT_, EPI_)                                                                          \
    e = cudaFuncSetAttribute(qkv_rope_append_kernel<BT_, EPI_>,                                    \
                             cudaFuncAttributeMaxDynamicSharedMemorySize,                          \
                             QkvSmem<BT_, row_blocks(EPI_)>::TOTAL);                               \
    if (e != cudaSuccess) return e;
    AC_SET(8, EPI_QKV_ROPE_APPEND)
    AC_SET(16, EPI_QKV_ROPE_APPEND)
    AC_SET(8, EPI_RESIDUAL_ADD)
    AC_SET(16, EPI_RESIDUAL_ADD)
    AC_SET(8, EPI_QKV_ROPE_VARIANT)
    AC_SET(16, EPI_QKV_ROPE_VARIANT)
#undef AC_SET
    return cudaSuccess;
}

// Batch rows per CTA tile.  The library sends batches above 16 rows to the tcgen05 kernels; this kernel
// would still serve them, 16 rows per grid slice.
int qkv_batch_tile(int B) { return B <= 8 ? 8 : 16; }

cudaError_t launch_qkv_rope_kv_append(const CUtensorMap& w_map, const CUtensorMap& x_map, void* q_out,
                                      void* k_cache, void* v_cache, int64_t stride_page,
                                      int64_t stride_token, int64_t stride_head,
                                      const int32_t* block_table, int max_pages_per_seq,
                                      const int32_t* context_lens, const float* rope_cos,
                                      const float* rope_sin, int max_position, int B, int H, int Hq,
                                      int Hkv, int d, int page_size, int num_pages, int32_t* status_flag,
                                      const RopeVariant* variant, cudaStream_t stream) {
    QkvParams p;
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
    p.H = H;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.d = d;
    p.residual_in = nullptr;
    p.residual_out = nullptr;
    p.N = 0;
    const int bt = qkv_batch_tile(B);
    p.rotary_dim = d;
    p.interleaved = 0;
    p.q_norm_w = p.k_norm_w = nullptr;
    p.norm_eps = 0.0f;
    if (variant != nullptr) {
        p.rotary_dim = variant->rotary_dim;
        p.interleaved = variant->interleaved;
        p.q_norm_w = static_cast<const uint16_t*>(variant->q_norm_weight);
        p.k_norm_w = static_cast<const uint16_t*>(variant->k_norm_weight);
        p.norm_eps = variant->norm_eps;
        if (bt == 8) return launch_qkv<8, EPI_QKV_ROPE_VARIANT>(w_map, x_map, p, stream);
        return launch_qkv<16, EPI_QKV_ROPE_VARIANT>(w_map, x_map, p, stream);
    }
    if (bt == 8) return launch_qkv<8, EPI_QKV_ROPE_APPEND>(w_map, x_map, p, stream);
    return launch_qkv<16, EPI_QKV_ROPE_APPEND>(w_map, x_map, p, stream);
}

// ---- RMSNorm of whole rows (second launch of the output-projection fusion) -------------------------
namespace {

// gridDim.x CTAs per row: each recomputes the row's sum of squares in fp64 (exact for bf16 inputs
// of moderate range, so every CTA gets the same value; the row is a few KB and sits in L2) and
// normalises its own slice: y = bf16(bf16(h / sqrt(mean + eps)) * w), the arithmetic of the per-head
// norm of the prelude.  Few rows are cut into up to eight slices so that the launch still covers the
// GPU; many rows need no slicing, and recomputing the sum eight times would only cost time.
constexpr int NORM_MAX_SLICES = 8;

__global__ void __launch_bounds__(256) rmsnorm_rows_kernel(const uint16_t* __restrict__ h,
                                                           const uint16_t* __restrict__ weight,
                                                           uint16_t* __restrict__ out, int N, float eps) {
    cudaTriggerProgrammaticLaunchCompletion();
    cudaGridDependencySynchronize();
    __shared__ double s_part[8];
    const uint16_t* row = h + static_cast<size_t>(blockIdx.y) * N;
    double ss = 0.0;
    for (int i = threadIdx.x * 8; i < N; i += 256 * 8) {          // N % 32 == 0: 16-byte pieces
        const uint4 v8 = *reinterpret_cast<const uint4*>(row + i);
        const uint32_t w4[4] = {v8.x, v8.y, v8.z, v8.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const double lo = static_cast<double>(__uint_as_float(w4[e] << 16));
            const double hi = static_cast<double>(__uint_as_float(w4[e] & 0xFFFF0000u));
            ss = __dadd_rn(ss, __dadd_rn(__dmul_rn(lo, lo), __dmul_rn(hi, hi)));
        }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) ss = __dadd_rn(ss, __shfl_xor_sync(0xffffffffu, ss, off));
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    double total = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) total = __dadd_rn(total, s_part[w]);
    const double r = __ddiv_rn(1.0, __dsqrt_rn(__dadd_rn(__ddiv_rn(total, static_cast<double>(N)),
                                                         static_cast<double>(eps))));
    uint16_t* orow = out + static_cast<size_t>(blockIdx.y) * N;
    const int per = (N + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    const int lo_i = blockIdx.x * per;
    const int hi_i = min(N, lo_i + per);
    for (int i = lo_i + threadIdx.x; i < hi_i; i += 256) {
        const double v = static_cast<double>(bf16_bits_to_float(row[i]));
        const uint16_t y1 = f64_to_bf16_rne(__dmul_rn(v, r));
        const double w = static_cast<double>(bf16_bits_to_float(weight[i]));
        orow[i] = f64_to_bf16_rne(__dmul_rn(static_cast<double>(bf16_bits_to_float(y1)), w));
    }
}

}  // namespace

cudaError_t launch_oproj_residual(const CUtensorMap& w_map, const CUtensorMap& x_map,
                                  const void* residual_in, void* residual_out, int B, int K, int N,
                                  cudaStream_t stream) {
    QkvParams p = {};
    p.B = B;
    p.H = K;
    p.N = N;
    p.residual_in = static_cast<const uint16_t*>(residual_in);
    p.residual_out = static_cast<uint16_t*>(residual_out);
    const int bt = qkv_batch_tile(B);
    if (bt == 8) return launch_qkv<8, EPI_RESIDUAL_ADD>(w_map, x_map, p, stream);
    return launch_qkv<16, EPI_RESIDUAL_ADD>(w_map, x_map, p, stream);
}

cudaError_t launch_rmsnorm_rows(const void* h, const void* weight, void* out, int B, int N, float eps,
                                cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    int slices = (2 * 148 + B - 1) / B;                 // about two CTAs per SM in total
    slices = slices < 1 ? 1 : (slices > NORM_MAX_SLICES ? NORM_MAX_SLICES : slices);
    cfg.gridDim = dim3(slices, B);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, rmsnorm_rows_kernel, static_cast<const uint16_t*>(h),
                              static_cast<const uint16_t*>(weight), static_cast<uint16_t*>(out), N, eps);
}

}  // namespace ac
