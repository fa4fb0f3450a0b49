// A4: single-token decode attention over a paged KV cache, one CTA per (request, KV head, split).
//
// Data movement.  The K and V pools are described to the TMA unit as 5-D tensors
// (64 elements, token-in-page, 64-element block of head_dim, head, page).  A work tile is 16
// consecutive tokens of one KV head inside one page: ONE box load [64 x 16 x head_dim/64] for K and
// one for V, which lands in shared memory as head_dim/64 blocks of [16 tokens x 128 bytes] with the
// 128-byte swizzle, so ldmatrix reads are free of bank conflicts.  (Issuing a tensor load costs the
// issuing thread on the order of 100 ns, so the number of loads per tile matters: splitting head_dim
// into the innermost 64 elements and an outer block index keeps the swizzle span at 128 bytes while
// still fetching the whole 256-byte rows with one instruction.)  Every warp runs its own ring of
// two tiles with one mbarrier per stage and takes tiles warp, warp+WARPS, ... of the CTA's token range
// (six warps per CTA and two CTAs per SM; twelve warps when the grid is at most one CTA per SM and
// the splits are long); there is no
// CTA-wide synchronisation in the main loop.  The physical page id of a tile is fetched from the block
// table one tile ahead of the TMA issue that needs it.  KV bytes are read once, so the loads carry an
// evict-first L2 policy.
//
// Arithmetic.  The Hq/Hkv query heads of the group are the rows of a 16-row MMA tile (rows >= group
// size are zero).  S = Q K^T and O += P V use the bf16 m16n8k16 warp MMA with fp32 accumulators; the
// accumulator layout of S is the A-operand layout of the second product, so P never leaves
// registers.  Softmax is the online form (running max and sum per row, in the exp2 domain) with
// warp-shuffle reductions across the four lanes that share a row.  At the end the warps' partial
// (max, sum, O) are combined through shared memory and the CTA writes either the final bf16 row
// (one split) or its normalised fp32 partial plus the natural-log log-sum-exp (several splits).
// With the fused merge the splits of a (request, KV head) are combined inside this kernel: by the CTA
// that arrives last (ticket on a global counter, partials through global memory), or, for grids of
// at most one CTA per SM, by the CTA of split 0 of a thread-block cluster that reads the other splits'
// results out of their shared memory.
//
// In the fused step (ROPE_PLAIN, ROPE_VARIANT) the kernel also rotates the new q and k -- with the plain
// rotate-half pairing, or with the prelude variants: per-head RMSNorm, partial rotary, interleaved
// pairing -- and appends k and v to the cache page before attending over them.
//
// With a group of 4-8 query rows the path needs G flop per KV byte; at HBM speed that exceeds what
// the fp32 pipes deliver for G >= 7, which is why the products run on the tensor pipe even though
// the kernel is bound by HBM bandwidth.
#include <limits.h>
#include <math.h>

#include "ac_device.cuh"
#include "ac_internal.h"
#include "rope_variant.cuh"

namespace ac {
namespace {

using namespace acdev;

constexpr int kWarps = 6;                     // warps per CTA, two CTAs per SM
constexpr int kFatWarps = 12;                 // warps per CTA when the SM holds one CTA (grids of at most one CTA per SM)
constexpr int kSlimWarps = 4;                 // warps per CTA, two CTAs per SM, for one wave of very long splits
constexpr int kSlimMinSplitTokens = 8192;
constexpr int kSlimMinWindowSplitTokens = 2048;
constexpr int kStages = 2;                    // tiles in flight per warp
constexpr int TILE = 16;                      // tokens per stage
constexpr int kLongestFirstMaxBatch = 128;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

template <int D, int NW>
struct Smem {
    static constexpr int STAGES = kStages;
    static constexpr int HALVES = D / 64;                 // 64-element (128-byte) column blocks
    static constexpr int HALF_BYTES = TILE * 128;         // one swizzled [16 x 128 B] block
    static constexpr int K_BYTES = HALVES * HALF_BYTES;   // K tile; V tile has the same size
    static constexpr int STAGE_BYTES = 2 * K_BYTES;
    static constexpr int RING_BYTES = STAGES * STAGE_BYTES;
    static constexpr int BAR_OFFSET = NW * RING_BYTES;
    static constexpr int TOTAL = BAR_OFFSET + NW * STAGES * 8 + 1024;      // + alignment slack
};

struct AttnParams {
    // -- only for the fused step (ROPE != ROPE_NONE): the kernel rotates q/k and appends k/v itself
    uint16_t* q_rot_out;          // [B, Hq, D] rotated q, optional (must not alias q)
    const uint16_t* k_new;        // [B, Hkv, D] un-rotated
    const uint16_t* v_new;        // [B, Hkv, D]
    uint16_t* k_cache;            // page pools (element strides below)
    uint16_t* v_cache;
    int64_t stride_page, stride_token, stride_head;
    const float* rope_cos;        // [max_position, D/2]
    const float* rope_sin;
    int max_position, num_pages;
    // -- always
    const uint16_t* q;            // [B, Hq, D] bf16: already rotated (ROPE_NONE) or raw (fused step)
    const int32_t* block_table;   // [B, max_pages_per_seq]
    const int32_t* context_lens;  // [B]
    float* partial_o;             // [B, Hq, S, D]   (S > 1)
    float* partial_lse;           // [B, Hq, S]      (S > 1)
    uint16_t* out;                // [B, Hq, D] bf16 (S == 1)
    uint16_t* out_mirror;         // optional second destination of every store to `out` (nullptr: none)
    int32_t* status_flag;
    int32_t* arrivals;            // [B, Hkv] arrival counters, zero on entry (fused merge only)
    float scale_log2;             // softmax scale * log2(e)
    int max_pages_per_seq;
    int new_tokens;
    int num_splits;
    int split_tokens;
    int Hq, Hkv, page_size;
    int fused_merge;              // 1: the last CTA of a (request, KV head) merges the splits itself
    const int32_t* row_order;     // optional [B] permutation: grid row y serves request row_order[y]
    int longest_first;            // 1: grid row y serves the request with the y-th longest context
    int window;                   // > 0: attend over the last `window` tokens of each row only
    int cluster_merge;            // 1: the splits of a (request, KV head) are one thread-block cluster and
                                  //    split 0 merges them out of the others' shared memory
    // -- only for the fused step with prelude variants (ROPE = 2)
    int rotary_dim;               // even, 2 .. D: elements [0, rotary_dim) rotate; tables are [max_position, rotary_dim/2]
    int interleaved;              // 0: pair (i, i + rotary_dim/2); 1: pair (2i, 2i + 1)
    const uint16_t* q_norm_w;     // bf16 [D] or nullptr: RMSNorm of every q head vector before the rotation
    const uint16_t* k_norm_w;     // same for k
    float norm_eps;
};

// Rotation flavours of the kernel: none (q arrives rotated), the plain rotate-half of the fused step,
// and the fused step with the prelude variants (per-head RMSNorm, partial rotary, interleaved pairing).
constexpr int ROPE_NONE = 0, ROPE_PLAIN = 1, ROPE_VARIANT = 2;

// The merge of the ticket path: the CTA that arrived last combines the splits' partial results of its
// (request, KV head) out of the workspace.  An item is four consecutive output elements of one query
// row; a thread owns ITEMS of them (item = thread + k * THREADS) and walks the splits in groups of GS
// for all its items at once: the ITEMS * GS 16-byte partial loads and their log-sum-exps are issued
// before any is used, so a group costs one L2 round trip whatever the number of items, and groups are
// combined with the same running-maximum rescaling as the main loop.  ITEMS * GS <= 16 keeps the
// loads in registers.
template <int D, int THREADS, int ITEMS, int GS>
__device__ __forceinline__ void merge_splits_from_workspace(const AttnParams& p, size_t hq0, int items, int S,
                                                            int n_active) {
    constexpr int D4 = D / 4;
    static_assert(ITEMS * GS <= 16, "loads of a group stay in registers");
    const float* lse_g[ITEMS];
    const float4* po[ITEMS];
    bool live[ITEMS];
    float M[ITEMS], den[ITEMS];
    float4 acc[ITEMS];
    size_t out_at[ITEMS];
#pragma unroll
    for (int k = 0; k < ITEMS; ++k) {
        const int e = threadIdx.x + k * THREADS;
        live[k] = e < items;
        const int row = live[k] ? e / D4 : 0;
        const int c4 = live[k] ? e - row * D4 : 0;
        lse_g[k] = p.partial_lse + (hq0 + row) * S;
        po[k] = reinterpret_cast<const float4*>(p.partial_o + (hq0 + row) * S * D) + c4;
        out_at[k] = (hq0 + row) * D + c4 * 4;
        M[k] = -INFINITY;
        den[k] = 0.0f;
        acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int s0 = 0; s0 < n_active; s0 += GS) {
        float4 v[ITEMS][GS];
        float l[ITEMS][GS];
#pragma unroll
        for (int k = 0; k < ITEMS; ++k)
#pragma unroll
            for (int u = 0; u < GS; ++u) {
                const bool on = live[k] && s0 + u < n_active;
                l[k][u] = on ? __ldcg(lse_g[k] + s0 + u) : -INFINITY;
                v[k][u] = on ? __ldcg(po[k] + static_cast<size_t>(s0 + u) * D4) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
        for (int k = 0; k < ITEMS; ++k) {
            float gm = M[k];
#pragma unroll
            for (int u = 0; u < GS; ++u) gm = fmaxf(gm, l[k][u]);
            const float rescale = __expf(M[k] - gm);           // 0 on the first group (M = -inf)
            acc[k].x *= rescale;
            acc[k].y *= rescale;
            acc[k].z *= rescale;
            acc[k].w *= rescale;
            den[k] *= rescale;
            M[k] = gm;
#pragma unroll
            for (int u = 0; u < GS; ++u) {
                const float wgt = __expf(l[k][u] - gm);        // 0 for the padding entries
                acc[k].x = fmaf(wgt, v[k][u].x, acc[k].x);
                acc[k].y = fmaf(wgt, v[k][u].y, acc[k].y);
                acc[k].z = fmaf(wgt, v[k][u].z, acc[k].z);
                acc[k].w = fmaf(wgt, v[k][u].w, acc[k].w);
                den[k] += wgt;
            }
        }
    }
#pragma unroll
    for (int k = 0; k < ITEMS; ++k) {
        if (!live[k]) continue;
        const float inv = 1.0f / den[k];
        const uint2 bits = make_uint2(pack_bf16x2(acc[k].x * inv, acc[k].y * inv),
                                      pack_bf16x2(acc[k].z * inv, acc[k].w * inv));
        *reinterpret_cast<uint2*>(p.out + out_at[k]) = bits;
        if (p.out_mirror != nullptr) *reinterpret_cast<uint2*>(p.out_mirror + out_at[k]) = bits;
    }
}

template <int D, bool WIDE, int ROPE, int NW>
__global__ void __launch_bounds__(NW * 32, NW == kFatWarps ? 1 : 2) paged_decode_attn_kernel(
    const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
    const AttnParams p) {
    using L = Smem<D, NW>;
    constexpr int WARPS = NW;
    constexpr int THREADS = NW * 32;
    constexpr int STAGES = kStages;
    constexpr int ROWS = WIDE ? 2 : 1;          // row blocks of 8 query heads held per thread
    constexpr int KSTEPS = D / 16;
    constexpr int NTILES = D / 8;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_addr(smem_raw));

    const int h = blockIdx.x;
    const int split = blockIdx.z;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    int b = blockIdx.y;
    if (p.row_order != nullptr) {
        // The caller (a scheduler that knows the lengths) supplied the order in which grid rows serve
        // requests, normally longest first.
        b = p.row_order[blockIdx.y];
    } else if (p.longest_first) {
        // The hardware hands out CTAs in grid order; when the grid is several waves deep, serving
        // the longest requests first keeps the short ones for the tail of the grid (greedy
        // longest-processing-time order).  Every CTA derives the same ranking from context_lens:
        // thread t counts the requests that sort before request t (longer, or equal and earlier).
        __shared__ int s_request;
        int* s_len = reinterpret_cast<int*>(smem_gen);            // the rings are not in use yet
        const int B = gridDim.y;
        const int B4 = (B + 3) & ~3;
        for (int i = threadIdx.x; i < B4; i += THREADS) s_len[i] = i < B ? p.context_lens[i] : INT_MIN;
        __syncthreads();
        for (int t = threadIdx.x; t < B; t += THREADS) {
            const int mine = s_len[t];
            int rank = 0;
            for (int j = 0; j < B4; j += 4) {               // padding entries never sort before anything
                const int4 o = *reinterpret_cast<const int4*>(s_len + j);
                rank += (o.x > mine) || (o.x == mine && j < t);
                rank += (o.y > mine) || (o.y == mine && j + 1 < t);
                rank += (o.z > mine) || (o.z == mine && j + 2 < t);
                rank += (o.w > mine) || (o.w == mine && j + 3 < t);
            }
            if (rank == static_cast<int>(blockIdx.y)) s_request = t;
        }
        __syncthreads();
        b = s_request;
    }
    const int G = p.Hq / p.Hkv;
    const int S = p.num_splits;

    // Everything up to the first read of q or of a cache slot that the preceding kernel may have
    // written is independent of that kernel, so with a programmatic dependent launch it overlaps the
    // preceding kernel's execution.  The preceding kernel is either the RoPE + append kernel of this
    // step (writes slot ctx) or the fused step of the previous token (wrote slot ctx - 1).
    int tok_begin = split * p.split_tokens;          // both move up when a sliding window applies
    int tile_begin = tok_begin / TILE;
    auto tile_token0 = [&](int j) { return (tile_begin + warp + j * WARPS) * TILE; };
    const int32_t* bt_row = p.block_table + static_cast<size_t>(b) * p.max_pages_per_seq;
    auto load_page_id = [&](int j) {
        const int idx = tile_token0(j) / p.page_size;
        return idx < p.max_pages_per_seq ? bt_row[idx] : -1;
    };

    const int ctx = p.context_lens[b];
    int page_first[STAGES];                       // page ids of the first tiles, fetched alongside ctx
#pragma unroll
    for (int s = 0; s < STAGES; ++s) page_first[s] = load_page_id(s);

    int n_tokens = ctx < 0 ? 0 : ctx + p.new_tokens;
    const long long table_tokens = static_cast<long long>(p.max_pages_per_seq) * p.page_size;
    if (n_tokens > table_tokens) n_tokens = static_cast<int>(table_tokens);
    // Sliding window: the row attends over tokens [tok_lo, n_tokens).  The splits partition the range
    // that starts at tok_lo rounded down to a multiple of 64; tiles wholly below tok_lo are skipped
    // and the first tile masks its leading tokens.
    int tok_lo = 0, window_base = 0;
    if (p.window > 0) {
        tok_lo = max(0, n_tokens - p.window);
        window_base = tok_lo / 64 * 64;
        tok_begin = max(window_base + split * p.split_tokens, tok_lo / TILE * TILE);
        tile_begin = tok_begin / TILE;
#pragma unroll
        for (int s = 0; s < STAGES; ++s) page_first[s] = load_page_id(s);     // the range moved
    }
    const int tok_end = min(window_base + (split + 1) * p.split_tokens, n_tokens);

    // Programmatic launch completion is signalled only AFTER this CTA has synchronised on the
    // preceding kernel (dependency_sync below).  The next kernel of the stream (launched with the
    // programmatic-serialization attribute, as the kernels of this library are) then becomes resident
    // while this grid is still running -- its set-up and first loads fill the SM slots that free up
    // during this grid's tail -- but never before the kernel ahead of this one has completed: at most
    // two kernels of a chain are in flight, so what a kernel reads before its own synchronisation can
    // only be stale with respect to its direct predecessor, which is what the tile limit below
    // (first_dependent_tile) accounts for.
    auto dependency_sync = [&]() {
        cudaGridDependencySynchronize();
        cudaTriggerProgrammaticLaunchCompletion();
    };

    if (tok_begin >= tok_end) {
        // Nothing to attend over in this split.  The buffers written here may still be in use by
        // the preceding kernel (a merge of the previous step, say), so wait for it first.
        dependency_sync();
        if (S > 1) {
            if (!p.fused_merge && threadIdx.x < G)
                p.partial_lse[(static_cast<size_t>(b) * p.Hq + h * G + threadIdx.x) * S + split] = -INFINITY;
            if (p.fused_merge && split == 0) {   // a row with no tokens at all: its output is +0
                const size_t o = (static_cast<size_t>(b) * p.Hq + h * G) * D;
                for (int e = threadIdx.x; e < G * D; e += THREADS) {
                    p.out[o + e] = 0;
                    if (p.out_mirror != nullptr) p.out_mirror[o + e] = 0;
                }
            }
        } else {
            const size_t o = (static_cast<size_t>(b) * p.Hq + h * G) * D;
            for (int e = threadIdx.x; e < G * D; e += THREADS) {
                p.out[o + e] = 0;
                if (p.out_mirror != nullptr) p.out_mirror[o + e] = 0;
            }
        }
        if (p.cluster_merge != 0 && S > 1) {
            // Cluster merge: keep step with the two cluster barriers of the CTAs that have tokens
            // (this CTA stages nothing and nobody reads its shared memory).
            cluster_sync_all();
            cluster_arrive_relaxed_all();
            cluster_wait_all();
        }
        return;
    }

    const uint32_t ring = smem_base + warp * L::RING_BYTES;
    const uint32_t bars = smem_base + L::BAR_OFFSET + warp * STAGES * 8;
    if (lane == 0) {
        tma_prefetch_descriptor(&k_map);
        tma_prefetch_descriptor(&v_map);
#pragma unroll
        for (int s = 0; s < STAGES; ++s) mbar_init(bars + s * 8, 1);
        mbar_init_fence();
    }
    __syncwarp();

    const int n_tiles = (tok_end - tok_begin + TILE - 1) / TILE;
    const int n_my = n_tiles > warp ? (n_tiles - warp + WARPS - 1) / WARPS : 0;
    const uint64_t policy = l2_policy_evict_first();
    // Tiles from the one holding slot ctx - 1 onwards must not be fetched before the preceding kernel
    // has completed; new_token_tile is where this step's own token lives.
    const int new_token_tile = p.new_tokens > 0 ? ctx / TILE : -1;
    const int first_dependent_tile = (ctx > 0 ? ctx - 1 : 0) / TILE;

    auto issue_at = [&](int j, int slot, int page) {      // lane 0 only; slot = first token's slot inside its page
        const int stage = j % STAGES;
        const uint32_t bar = bars + stage * 8;
        const uint32_t dst = ring + stage * L::STAGE_BYTES;
        mbar_arrive_expect_tx(bar, L::STAGE_BYTES);
        tma_load_5d(dst, &k_map, bar, 0, slot, 0, h, page, policy);
        tma_load_5d(dst + L::K_BYTES, &v_map, bar, 0, slot, 0, h, page, policy);
    };

    // Fused step: the rotary angles of this CTA's query rows depend only on ctx; fetch them now so
    // that they are in registers when q itself can be read (after the dependency is met).
    constexpr int QP = ROPE == ROPE_PLAIN ? (16 * (D / 2) + THREADS - 1) / THREADS : 1;   // rotary pairs per thread
    // The new token can be appended only if its position has a rope-table row, a block-table entry
    // and a tile in this launch's split grid (max_context_len too small for the row otherwise).
    const bool rope_ok = ROPE && ctx < p.max_position &&
                         ctx < table_tokens &&
                         static_cast<long long>(ctx) <
                             window_base + static_cast<long long>(S) * p.split_tokens;
    float q_cos[QP], q_sin[QP];
    if (ROPE == ROPE_PLAIN) {
        const float* cos_row = p.rope_cos + static_cast<size_t>(ctx) * (D / 2);
        const float* sin_row = p.rope_sin + static_cast<size_t>(ctx) * (D / 2);
#pragma unroll
        for (int k = 0; k < QP; ++k) {
            const int idx = threadIdx.x + k * THREADS;
            const int row = idx / (D / 2);
            const int i = idx - row * (D / 2);
            const bool on = rope_ok && row < G;
            q_cos[k] = on ? cos_row[i] : 1.0f;
            q_sin[k] = on ? sin_row[i] : 0.0f;
        }
    }

    // ---- prologue: fill the ring -------------------------------------------------------------
    int issued = 0;
    bool dependency_met = false;
#pragma unroll
    for (int s = 0; s < STAGES; ++s) {
        if (s < n_my) {
            if (!dependency_met && tile_begin + warp + s * WARPS >= first_dependent_tile) {
                dependency_sync();
                dependency_met = true;
            }
            if (lane == 0) issue_at(s, tile_token0(s) % p.page_size, page_first[s]);
            issued = s + 1;
        }
    }
    int page_next = issued < n_my ? load_page_id(issued) : 0;
    // Where this warp's next tile sits in the row (block-table index, slot inside the page).  A warp's
    // tiles are WARPS * TILE tokens apart, so from here on the position is stepped, not divided: the two
    // integer divisions by the run-time page size per refill cost a fifth of a warp's time per tile.
    const int step_tokens = WARPS * TILE;
    const int step_pages = step_tokens / p.page_size, step_slots = step_tokens - step_pages * p.page_size;
    int next_idx = tile_token0(issued) / p.page_size;
    int next_slot = tile_token0(issued) - next_idx * p.page_size;
    if (!dependency_met) dependency_sync();                    // q was written by the preceding kernel
    uint16_t q_raw_lo[QP], q_raw_hi[QP];
    if (ROPE == ROPE_PLAIN) {
        const uint16_t* qsrc = p.q + (static_cast<size_t>(b) * p.Hq + h * G) * D;
#pragma unroll
        for (int k = 0; k < QP; ++k) {
            const int idx = threadIdx.x + k * THREADS;
            const int row = idx / (D / 2);
            const int i = idx - row * (D / 2);
            const bool on = row < G;
            q_raw_lo[k] = on ? qsrc[row * D + i] : static_cast<uint16_t>(0);
            q_raw_hi[k] = on ? qsrc[row * D + i + D / 2] : static_cast<uint16_t>(0);
        }
    }

    // ---- fused step: rotate and append the new k/v early, under the latency of the first tiles ------
    constexpr int APPEND_PAIRS = D / 64;          // rotary pairs per lane (D/2 pairs over 32 lanes)
    constexpr int EPL = D / 32;                   // variants: lane l holds elements l*EPL .. l*EPL + EPL - 1
    uint16_t k_rot_lo[APPEND_PAIRS], k_rot_hi[APPEND_PAIRS];
    uint16_t k_var[EPL];
    __shared__ uint16_t s_kpark[ROPE == ROPE_VARIANT ? D : 8];     // the appending warp's parked k vector
    uint2 v_new4 = make_uint2(0u, 0u);
    int append_j = -1;                            // index of this warp's tile that holds the new slot
    bool append_ok = false;
    if (ROPE) {
        if (!rope_ok && threadIdx.x == 0 && p.status_flag != nullptr)
            atomicOr(p.status_flag, AC_FLAG_POSITION_OOB);
        const int rel = new_token_tile - tile_begin - warp;
        if (rel >= 0 && rel % WARPS == 0 && rel / WARPS < n_my) append_j = rel / WARPS;
        if (append_j >= 0 && rope_ok) {
            const int page = load_page_id(append_j);
            if (page < 0 || page >= p.num_pages) {
                if (lane == 0 && p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_PAGE_OOB);
            } else {
                append_ok = true;
                const size_t goff = static_cast<size_t>(page) * p.stride_page +
                                    static_cast<size_t>(ctx % p.page_size) * p.stride_token +
                                    static_cast<size_t>(h) * p.stride_head;
                const uint16_t* ksrc = p.k_new + (static_cast<size_t>(b) * p.Hkv + h) * D;
                const uint16_t* vsrc = p.v_new + (static_cast<size_t>(b) * p.Hkv + h) * D;
                if (ROPE == ROPE_VARIANT) {
                    const int half_r = p.rotary_dim / 2;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) k_var[e] = ksrc[lane * EPL + e];
                    rope_variant_vector<D>(k_var, p.k_norm_w, p.norm_eps,
                                           p.rope_cos + static_cast<size_t>(ctx) * half_r,
                                           p.rope_sin + static_cast<size_t>(ctx) * half_r, p.rotary_dim,
                                           p.interleaved, s_kpark, lane);
#pragma unroll
                    for (int e = 0; e < EPL; ++e) p.k_cache[goff + lane * EPL + e] = k_var[e];
                } else {
                    const float* cos_row = p.rope_cos + static_cast<size_t>(ctx) * (D / 2);
                    const float* sin_row = p.rope_sin + static_cast<size_t>(ctx) * (D / 2);
#pragma unroll
                    for (int u = 0; u < APPEND_PAIRS; ++u) {
                        const int i = lane + 32 * u;
                        const uint16_t a = ksrc[i], bb = ksrc[i + D / 2];
                        const float c = cos_row[i], sn = sin_row[i];
                        k_rot_lo[u] = rope_first_half(a, bb, c, sn);
                        k_rot_hi[u] = rope_second_half(a, bb, c, sn);
                        p.k_cache[goff + i] = k_rot_lo[u];
                        p.k_cache[goff + i + D / 2] = k_rot_hi[u];
                    }
                }
                if (lane * 4 < D) {
                    v_new4 = *reinterpret_cast<const uint2*>(vsrc + lane * 4);
                    *reinterpret_cast<uint2*>(p.v_cache + goff + lane * 4) = v_new4;
                }
            }
        }
    }

    // ---- query fragments (A operand of Q K^T), rows = heads of the group ---------------------------
    const int g = lane >> 2;
    const int t = lane & 3;
    uint32_t qa[KSTEPS][2 * ROWS];
    constexpr int QSTRIDE = D + 8;                 // padded row: fragment loads hit 32 distinct banks
    __shared__ __align__(16) uint16_t s_q[ROPE ? 16 * QSTRIDE : 8];
    if (ROPE == ROPE_VARIANT) {
        // Prelude variants: one warp per query row (rows warp, warp + 6, ...): optional RMSNorm, then the
        // partial / interleaved rotation, with the row's place in the shared tile as the parking space
        // for the partner look-ups.  Same arithmetic as the stand-alone variant kernel.
        uint16_t* qdst = (p.q_rot_out != nullptr && split == 0)
                             ? p.q_rot_out + (static_cast<size_t>(b) * p.Hq + h * G) * D : nullptr;
        const uint16_t* qsrc = p.q + (static_cast<size_t>(b) * p.Hq + h * G) * D;
        const int half_r = p.rotary_dim / 2;
        for (int row = warp; row < (WIDE ? 16 : 8); row += WARPS) {
            uint16_t xq[EPL];
#pragma unroll
            for (int e = 0; e < EPL; ++e) xq[e] = row < G ? qsrc[row * D + lane * EPL + e] : static_cast<uint16_t>(0);
            if (row < G && rope_ok) {
                rope_variant_vector<D>(xq, p.q_norm_w, p.norm_eps, p.rope_cos + static_cast<size_t>(ctx) * half_r,
                                       p.rope_sin + static_cast<size_t>(ctx) * half_r, p.rotary_dim, p.interleaved,
                                       s_q + row * QSTRIDE, lane);
                if (qdst != nullptr) {
#pragma unroll
                    for (int e = 0; e < EPL; ++e) qdst[row * D + lane * EPL + e] = xq[e];
                }
            }
#pragma unroll
            for (int e = 0; e < EPL; ++e) s_q[row * QSTRIDE + lane * EPL + e] = xq[e];
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
            const int col = kk * 16 + 2 * t;
            qa[kk][0] = *reinterpret_cast<const uint32_t*>(s_q + g * QSTRIDE + col);
            qa[kk][ROWS] = *reinterpret_cast<const uint32_t*>(s_q + g * QSTRIDE + col + 8);
            if (WIDE) {
                qa[kk][1] = *reinterpret_cast<const uint32_t*>(s_q + (g + 8) * QSTRIDE + col);
                qa[kk][ROWS + 1] = *reinterpret_cast<const uint32_t*>(s_q + (g + 8) * QSTRIDE + col + 8);
            }
        }
    } else if (ROPE) {
        // The CTA rotates its G query rows once (pair i with i + D/2, exact then rounded, as the
        // stand-alone kernel does) into shared memory; every warp then reads its fragments from there.
        uint16_t* qdst = (p.q_rot_out != nullptr && split == 0)
                             ? p.q_rot_out + (static_cast<size_t>(b) * p.Hq + h * G) * D : nullptr;
#pragma unroll
        for (int k = 0; k < QP; ++k) {
            const int idx = threadIdx.x + k * THREADS;
            if (idx >= 16 * (D / 2)) break;
            const int row = idx / (D / 2);
            const int i = idx - row * (D / 2);
            uint16_t r0 = 0, r1 = 0;
            if (row < G) {
                if (rope_ok) {
                    r0 = rope_first_half(q_raw_lo[k], q_raw_hi[k], q_cos[k], q_sin[k]);
                    r1 = rope_second_half(q_raw_lo[k], q_raw_hi[k], q_cos[k], q_sin[k]);
                } else {
                    r0 = q_raw_lo[k];
                    r1 = q_raw_hi[k];
                }
                if (qdst != nullptr && rope_ok) {
                    qdst[row * D + i] = r0;
                    qdst[row * D + i + D / 2] = r1;
                }
            }
            if (WIDE || row < 8) {
                s_q[row * QSTRIDE + i] = r0;
                s_q[row * QSTRIDE + i + D / 2] = r1;
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
            const int col = kk * 16 + 2 * t;
            qa[kk][0] = *reinterpret_cast<const uint32_t*>(s_q + g * QSTRIDE + col);
            qa[kk][ROWS] = *reinterpret_cast<const uint32_t*>(s_q + g * QSTRIDE + col + 8);
            if (WIDE) {
                qa[kk][1] = *reinterpret_cast<const uint32_t*>(s_q + (g + 8) * QSTRIDE + col);
                qa[kk][ROWS + 1] = *reinterpret_cast<const uint32_t*>(s_q + (g + 8) * QSTRIDE + col + 8);
            }
        }
    } else {
        const uint16_t* qrow0 = p.q + (static_cast<size_t>(b) * p.Hq + h * G + g) * D;
        const bool v0 = g < G;
        const bool v1 = WIDE && (g + 8 < G);
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
            const int col = kk * 16 + 2 * t;
            qa[kk][0] = v0 ? *reinterpret_cast<const uint32_t*>(qrow0 + col) : 0u;
            qa[kk][ROWS] = v0 ? *reinterpret_cast<const uint32_t*>(qrow0 + col + 8) : 0u;
            if (WIDE) {
                qa[kk][1] = v1 ? *reinterpret_cast<const uint32_t*>(qrow0 + 8 * D + col) : 0u;
                qa[kk][ROWS + 1] = v1 ? *reinterpret_cast<const uint32_t*>(qrow0 + 8 * D + col + 8) : 0u;
            }
        }
    }
    // qa[kk] = {a0 (row g, k lo), [a1 (row g+8, k lo)], a2 (row g, k hi), [a3 (row g+8, k hi)]}

    float o[NTILES][2 * ROWS];
#pragma unroll
    for (int nt = 0; nt < NTILES; ++nt)
#pragma unroll
        for (int e = 0; e < 2 * ROWS; ++e) o[nt][e] = 0.0f;
    float m_run[ROWS], l_run[ROWS];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
        m_run[r] = -INFINITY;
        l_run[r] = 0.0f;
    }

    // lane-dependent parts of the ldmatrix addresses (row r of matrix mi; 128-byte rows, swizzled)
    const int mi = lane >> 3;
    const int r8 = lane & 7;
    const uint32_t k_row_off = ((mi >> 1) * 8 + r8) * 128;     // K: matrices 0,1 -> tokens 0-7; 2,3 -> 8-15
    const int k_chunk_lo = mi & 1;                              //    matrices 0,2 -> k lo; 1,3 -> k hi
    const uint32_t v_row_off = ((mi & 1) * 8 + r8) * 128;      // V: matrices 0,2 -> tokens 0-7; 1,3 -> 8-15
    const int v_chunk_lo = mi >> 1;                             //    matrices 0,1 -> n-tile even; 2,3 -> odd

    bool timed_out = false;
    int j = 0;
    for (; j < n_my; ++j) {
        const int stage = j % STAGES;
        const uint32_t kbase = ring + stage * L::STAGE_BYTES;
        const uint32_t vbase = kbase + L::K_BYTES;
        if (!mbar_wait_bounded(bars + stage * 8, (j / STAGES) & 1)) {
            timed_out = true;
            break;
        }
        bool wrote_stage = false;                              // ordinary stores went into this stage
        const int tok0 = tile_token0(j);
        const int n_valid = tok_end - tok0;                    // >= 1; < 16 only on the last tile
        const int lo_valid = tok_lo - tok0;                    // > 0 only on the first tile of a window

        if (ROPE && j == append_j && append_ok) {
            // The tile just loaded still has the stale slot of the new token: overwrite that row with
            // the rotated k and the v computed (and written to the cache) during the prologue.
            const int slot_in_tile = ctx - tok0;
            auto tile_byte = [&](int col) {       // byte offset of (slot_in_tile, col) inside a K or V tile
                return (col >> 6) * L::HALF_BYTES + slot_in_tile * 128 +
                       ((((col & 63) >> 3) ^ (slot_in_tile & 7)) << 4) + ((col & 7) << 1);
            };
            if (ROPE == ROPE_VARIANT) {
#pragma unroll
                for (int e = 0; e < EPL; ++e)
                    *reinterpret_cast<uint16_t*>(smem_gen + (kbase - smem_base) + tile_byte(lane * EPL + e)) = k_var[e];
            } else {
#pragma unroll
                for (int u = 0; u < APPEND_PAIRS; ++u) {
                    const int i = lane + 32 * u;
                    *reinterpret_cast<uint16_t*>(smem_gen + (kbase - smem_base) + tile_byte(i)) = k_rot_lo[u];
                    *reinterpret_cast<uint16_t*>(smem_gen + (kbase - smem_base) + tile_byte(i + D / 2)) = k_rot_hi[u];
                }
            }
            if (lane * 4 < D)
                *reinterpret_cast<uint2*>(smem_gen + (vbase - smem_base) + tile_byte(lane * 4)) = v_new4;
            wrote_stage = true;
            __syncwarp();
        }

        // ---- S = Q K^T for 16 tokens -------------------------------------------------------
        float s[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) s[nt][e] = 0.0f;
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
            const int dc = 2 * kk + k_chunk_lo;                // 16-byte column chunk of head_dim
            const uint32_t addr = kbase + (dc >> 3) * L::HALF_BYTES + k_row_off + (((dc & 7) ^ r8) << 4);
            uint32_t b00, b01, b10, b11;
            ldmatrix_x4(b00, b01, b10, b11, addr);
            if (WIDE) {
                mma_bf16_16816(s[0][0], s[0][1], s[0][2], s[0][3], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b00, b01);
                mma_bf16_16816(s[1][0], s[1][1], s[1][2], s[1][3], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b10, b11);
            } else {
                mma_bf16_16816_top(s[0][0], s[0][1], qa[kk][0], qa[kk][1], b00, b01);
                mma_bf16_16816_top(s[1][0], s[1][1], qa[kk][0], qa[kk][1], b10, b11);
            }
        }

        if (n_valid < TILE || lo_valid > 0) {
            // Slots past the request's length hold arbitrary bits, and tokens before a sliding
            // window's start are not attended: mask their scores and clear their V rows (0 * NaN
            // would poison the product).
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col = nt * 8 + 2 * t + (e & 1);
                    if (col >= n_valid || col < lo_valid) s[nt][e] = -INFINITY;
                }
            const int chunks_per_row = L::HALVES * 8;
            for (int idx = lane; idx < TILE * chunks_per_row; idx += 32) {
                const int row = idx / chunks_per_row;
                const int rem = idx % chunks_per_row;
                if (row >= n_valid || row < lo_valid) {
                    uint4* dstz = reinterpret_cast<uint4*>(smem_gen + (vbase - smem_base) +
                                                           (rem >> 3) * L::HALF_BYTES + row * 128 + (rem & 7) * 16);
                    *dstz = make_uint4(0u, 0u, 0u, 0u);
                }
            }
            wrote_stage = true;
            __syncwarp();
        }

        // ---- online softmax (exp2 domain) --------------------------------------------------
        uint32_t pa[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            float mx = fmaxf(fmaxf(s[0][2 * r], s[0][2 * r + 1]), fmaxf(s[1][2 * r], s[1][2 * r + 1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[r], mx * p.scale_log2);
            const float alpha = exp2f(m_run[r] - m_new);
            m_run[r] = m_new;
            const float p00 = exp2f(fmaf(s[0][2 * r], p.scale_log2, -m_new));
            const float p01 = exp2f(fmaf(s[0][2 * r + 1], p.scale_log2, -m_new));
            const float p10 = exp2f(fmaf(s[1][2 * r], p.scale_log2, -m_new));
            const float p11 = exp2f(fmaf(s[1][2 * r + 1], p.scale_log2, -m_new));
            l_run[r] = fmaf(l_run[r], alpha, (p00 + p01) + (p10 + p11));
            pa[r] = pack_bf16x2(p00, p01);          // a0 / a1: tokens 2t, 2t+1
            pa[2 + r] = pack_bf16x2(p10, p11);      // a2 / a3: tokens 2t+8, 2t+9
            if (alpha != 1.0f) {
#pragma unroll
                for (int nt = 0; nt < NTILES; ++nt) {
                    o[nt][2 * r] *= alpha;
                    o[nt][2 * r + 1] *= alpha;
                }
            }
        }

        // ---- O += P V ----------------------------------------------------------------------
#pragma unroll
        for (int jj = 0; jj < NTILES / 2; ++jj) {
            const int dc = 2 * jj + v_chunk_lo;
            const uint32_t addr = vbase + (dc >> 3) * L::HALF_BYTES + v_row_off + (((dc & 7) ^ r8) << 4);
            uint32_t b00, b01, b10, b11;
            ldmatrix_x4_trans(b00, b01, b10, b11, addr);
            if (WIDE) {
                mma_bf16_16816(o[2 * jj][0], o[2 * jj][1], o[2 * jj][2], o[2 * jj][3], pa[0], pa[1], pa[2], pa[3], b00, b01);
                mma_bf16_16816(o[2 * jj + 1][0], o[2 * jj + 1][1], o[2 * jj + 1][2], o[2 * jj + 1][3], pa[0], pa[1], pa[2], pa[3], b10, b11);
            } else {
                mma_bf16_16816_top(o[2 * jj][0], o[2 * jj][1], pa[0], pa[2], b00, b01);
                mma_bf16_16816_top(o[2 * jj + 1][0], o[2 * jj + 1][1], pa[0], pa[2], b10, b11);
            }
        }

        // ---- refill this stage -----------------------------------------------------------------
        // Ordinary (generic-proxy) stores into the stage -- the patch of the new token, the cleared V
        // rows of a ragged tile -- are ordered before the TMA (async-proxy) write that refills it.
        if (wrote_stage) fence_proxy_async_shared();
        __syncwarp();
        if (issued < n_my) {
            const int page = page_next;
            const int slot = next_slot;
            next_idx += step_pages;
            next_slot += step_slots;
            if (next_slot >= p.page_size) {
                next_slot -= p.page_size;
                ++next_idx;
            }
            page_next = issued + 1 < n_my ? (next_idx < p.max_pages_per_seq ? bt_row[next_idx] : -1) : 0;
            if (lane == 0) issue_at(issued, slot, page);
            ++issued;
        }
    }

    if (timed_out) {
        // Record the failure, then give the copies still in flight a bounded chance to land before
        // this CTA's shared memory is released.
        if (lane == 0 && p.status_flag != nullptr) atomicOr(p.status_flag, AC_FLAG_WAIT_TIMEOUT);
        for (int jj = j; jj < issued; ++jj) mbar_wait_bounded(bars + (jj % STAGES) * 8, (jj / STAGES) & 1);
    }

    // ---- combine the warps' partial results through shared memory ----------------------------------
    // Each warp reuses the start of its own ring (all of its loads have completed).
    constexpr int WROWS = 8 * ROWS;
    constexpr int WSTRIDE = D + 8;            // +8 floats: the 8-byte stores of a half-warp hit 32 banks
    float* wo = reinterpret_cast<float*>(smem_gen + warp * L::RING_BYTES);     // [WROWS][WSTRIDE]
    float* wm = wo + WROWS * WSTRIDE;                                           // [WROWS]
    float* wl = wm + WROWS;                                                     // [WROWS]
    static_assert((WROWS * WSTRIDE + 2 * WROWS) * 4 <= L::RING_BYTES, "merge scratch must fit in a ring");
    // Cluster merge: this CTA's normalised result is staged behind the warps' scratch, eight query rows
    // per ring (rows 0-7 in ring 0, rows 8-15 in ring 1): [8][D] fp32, then the 8 log-sum-exps.
    constexpr int STAGE_OFF = (WROWS * WSTRIDE + 2 * WROWS) * 4;
    static_assert(STAGE_OFF % 16 == 0 && STAGE_OFF + 8 * D * 4 + 8 * 4 <= L::RING_BYTES, "staged result must fit");
    auto staged_o = [&](int row, int col) {       // byte offset from smem_base
        return static_cast<uint32_t>((row >> 3) * L::RING_BYTES + STAGE_OFF + ((row & 7) * D + col) * 4);
    };
    auto staged_lse = [&](int row) {
        return static_cast<uint32_t>((row >> 3) * L::RING_BYTES + STAGE_OFF + 8 * D * 4 + (row & 7) * 4);
    };
    const bool cluster_merge = p.cluster_merge != 0 && S > 1;
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
        float l = l_run[r];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        const int row = g + 8 * r;
        if (t == 0) {
            wm[row] = m_run[r];
            wl[row] = l;
        }
#pragma unroll
        for (int nt = 0; nt < NTILES; ++nt)
            *reinterpret_cast<float2*>(wo + row * WSTRIDE + nt * 8 + 2 * t) = make_float2(o[nt][2 * r], o[nt][2 * r + 1]);
    }
    __syncthreads();

    // One item = four consecutive output elements of one query row: a warp covers one row per pass, so
    // the weights of the row's four partial results are computed once per item and reused for its four
    // columns, and every load and store is 16 bytes (8 for the bf16 result) wide.
    constexpr int C4 = D / 4;
    constexpr int PASSES = (WROWS * C4 + THREADS - 1) / THREADS;   // two or three: unrolled, their loads overlap
#pragma unroll
    for (int pass = 0; pass < PASSES; ++pass) {
        const int e = threadIdx.x + pass * THREADS;
        if (e >= G * C4) break;
        const int row = e / C4;
        const int col = (e - row * C4) * 4;
        float mw[WARPS];
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) {
            mw[w] = reinterpret_cast<const float*>(smem_gen + w * L::RING_BYTES)[WROWS * WSTRIDE + row];
            M = fmaxf(M, mw[w]);
        }
        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
        float den = 0.0f;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) {
            const float* base = reinterpret_cast<const float*>(smem_gen + w * L::RING_BYTES);
            const float wgt = exp2f(mw[w] - M);                 // 0 for a warp that saw no tile
            const float4 o4 = *reinterpret_cast<const float4*>(base + row * WSTRIDE + col);
            num.x = fmaf(wgt, o4.x, num.x);
            num.y = fmaf(wgt, o4.y, num.y);
            num.z = fmaf(wgt, o4.z, num.z);
            num.w = fmaf(wgt, o4.w, num.w);
            den = fmaf(wgt, base[WROWS * WSTRIDE + WROWS + row], den);
        }
        const float4 val = make_float4(num.x / den, num.y / den, num.z / den, num.w / den);
        const size_t hq = static_cast<size_t>(b) * p.Hq + h * G + row;
        if (S == 1) {
            const uint2 bits = make_uint2(pack_bf16x2(val.x, val.y), pack_bf16x2(val.z, val.w));
            *reinterpret_cast<uint2*>(p.out + hq * D + col) = bits;
            if (p.out_mirror != nullptr) *reinterpret_cast<uint2*>(p.out_mirror + hq * D + col) = bits;
        } else if (cluster_merge) {
            *reinterpret_cast<float4*>(smem_gen + staged_o(row, col)) = val;
            if (col == 0) *reinterpret_cast<float*>(smem_gen + staged_lse(row)) = (M + log2f(den)) * LN2;
        } else {
            *reinterpret_cast<float4*>(p.partial_o + (hq * S + split) * D + col) = val;
            if (col == 0) p.partial_lse[hq * S + split] = (M + log2f(den)) * LN2;
        }
    }

    if (S == 1 || !p.fused_merge) return;

    if (cluster_merge) {
        // ---- fused merge inside a cluster: split 0 reads the other splits' staged results out of
        // their shared memory.  No global round trip, no ticket; CTAs whose split has no tokens pass
        // through the same two barriers and nothing else.
        // splits with tokens, <= 16 (a row longer than the split grid covers still has S of them)
        const int n_active = min(S, (n_tokens - window_base + p.split_tokens - 1) / p.split_tokens);
        cluster_sync_all();                              // every staged result is written and visible
        if (split == 0) {
            constexpr int D4 = D / 4;
            const size_t hq0 = static_cast<size_t>(b) * p.Hq + h * G;
            for (int e = threadIdx.x; e < G * D4; e += THREADS) {
                const int row = e / D4;
                const int c4 = e - row * D4;
                const uint32_t o_addr = smem_base + staged_o(row, c4 * 4);
                const uint32_t l_addr = smem_base + staged_lse(row);
                float4 v[16];
                float l[16];
#pragma unroll
                for (int u = 0; u < 16; ++u) {           // all loads first: one round trip
                    const bool on = u < n_active;
                    l[u] = on ? cluster_load_f32(cluster_map_shared(l_addr, u)) : -INFINITY;
                    v[u] = on ? cluster_load_f32x4(cluster_map_shared(o_addr, u)) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                float M = -INFINITY;
#pragma unroll
                for (int u = 0; u < 16; ++u) M = fmaxf(M, l[u]);
                float den = 0.0f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    const float wgt = __expf(l[u] - M);  // 0 for the padding entries
                    acc.x = fmaf(wgt, v[u].x, acc.x);
                    acc.y = fmaf(wgt, v[u].y, acc.y);
                    acc.z = fmaf(wgt, v[u].z, acc.z);
                    acc.w = fmaf(wgt, v[u].w, acc.w);
                    den += wgt;
                }
                const float inv = 1.0f / den;
                const uint2 bits = make_uint2(pack_bf16x2(acc.x * inv, acc.y * inv), pack_bf16x2(acc.z * inv, acc.w * inv));
                *reinterpret_cast<uint2*>(p.out + (hq0 + row) * D + c4 * 4) = bits;
                if (p.out_mirror != nullptr) *reinterpret_cast<uint2*>(p.out_mirror + (hq0 + row) * D + c4 * 4) = bits;
            }
        }
        // Second barrier, in two halves and without a release: it publishes nothing, it only keeps every
        // CTA's shared memory alive until split 0 has consumed it (the values are in its registers by
        // then), so nobody waits for the result stores above to become visible.
        cluster_arrive_relaxed_all();
        cluster_wait_all();
        return;
    }

    // ---- fused merge: the CTA that arrives last for this (request, KV head) combines the splits ----
    // Publish this CTA's partials, take a ticket, and let the holder of the last ticket do the merge.
    // Nobody waits for anybody: CTAs that are not last simply exit.
    __shared__ int s_is_last;
    // splits with tokens (a row longer than the split grid covers still has S of them)
    const int n_active = min(S, (n_tokens - window_base + p.split_tokens - 1) / p.split_tokens);
    // One acquire-release atomic by one thread, bracketed by CTA barriers: the release orders the
    // partials that every thread of this CTA stored before the first barrier ahead of the ticket, the
    // acquire orders the ticket ahead of the partial loads that follow the second barrier.
    __syncthreads();
    if (threadIdx.x == 0) {
        int32_t* counter = p.arrivals + static_cast<size_t>(b) * p.Hkv + h;
        int ticket;
        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(ticket) : "l"(counter) : "memory");
        s_is_last = ticket == n_active - 1;
        if (s_is_last) *counter = 0;             // leave the counter ready for the next launch
    }
    __syncthreads();
    if (!s_is_last) return;
    const size_t hq0 = static_cast<size_t>(b) * p.Hq + h * G;
    const int items = G * (D / 4);                   // a thread owns up to three of them
    if (items <= THREADS) merge_splits_from_workspace<D, THREADS, 1, 16>(p, hq0, items, S, n_active);
    else if (items <= 2 * THREADS) merge_splits_from_workspace<D, THREADS, 2, 8>(p, hq0, items, S, n_active);
    else merge_splits_from_workspace<D, THREADS, 3, 5>(p, hq0, items, S, n_active);
}

template <int D, bool WIDE, int ROPE, int NW>
cudaError_t launch_one_staged(const CUtensorMap& k_map, const CUtensorMap& v_map, const AttnParams& p_in, int B,
                       cudaStream_t stream) {
    AttnParams p = p_in;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.Hkv, B, p.num_splits);
    cfg.blockDim = dim3(NW * 32);
    cfg.dynamicSmemBytes = Smem<D, NW>::TOTAL;
    cfg.stream = stream;
    // Programmatic dependent launch: this kernel may start while the preceding kernel of the
    // stream is still running; it calls cudaGridDependencySynchronize() before touching anything
    // that kernel produces.
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;    // the splits of a (request, KV head)
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = static_cast<unsigned>(p.num_splits);
    cfg.attrs = attr;
    if (p.cluster_merge) {
        // A cluster is placed inside one GPC, so fewer clusters than CTA slots / cluster size may be
        // resident at once (9-CTA clusters: 28 on a 148-SM part, not 32).  The cluster merge is used
        // only when every cluster of the grid is resident together; the answer per split count is
        // asked of the runtime once and remembered (benign race: every thread stores the same value).
        static int max_clusters[kMaxDevices][kClusterMergeMaxSplits + 1];     // 0 = not asked yet
        int dev = 0;
        cudaGetDevice(&dev);
        int& known = max_clusters[dev < kMaxDevices ? dev : 0][p.num_splits];
        if (known == 0) {
            int n = 0;
            cfg.numAttrs = 2;
            const cudaError_t qe = cudaOccupancyMaxActiveClusters(&n, paged_decode_attn_kernel<D, WIDE, ROPE, NW>, &cfg);
            if (qe != cudaSuccess) {
                cudaGetLastError();
                n = 0;
            }
            known = n > 0 ? n : -1;
        }
        if (static_cast<long long>(B) * p.Hkv > known) p.cluster_merge = 0;
    }
    cfg.numAttrs = p.cluster_merge ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, paged_decode_attn_kernel<D, WIDE, ROPE, NW>, k_map, v_map, p);
}

// Grids of at most one CTA per SM leave half of each SM's shared memory and warp slots unused: when a
// split holds more tiles than the six two-stage rings take at once, they run with twelve warps per CTA
// (the same bytes in flight per SM as two resident CTAs, and twice the warps to hide a warp's
// latency-bound time per tile).  Shorter splits keep the small footprint, which lets the next kernel of
// a chain become resident beside this one.
template <int D, bool WIDE, int ROPE>
cudaError_t launch_one(const CUtensorMap& k_map, const CUtensorMap& v_map, const AttnParams& p, int B,
                       cudaStream_t stream) {
    int dev = 0;
    cudaGetDevice(&dev);
    const long long ctas = static_cast<long long>(B) * p.Hkv * p.num_splits;
    const int sms = device_state(dev).sm_count;
    const bool fat = ctas <= sms && p.split_tokens > kStages * kWarps * TILE;
    if (fat) return launch_one_staged<D, WIDE, ROPE, kFatWarps>(k_map, v_map, p, B, stream);
    // One wave of very long splits, two CTAs per SM: every CTA streams for the whole launch, nothing
    // ramps beside it, and HBM delivers more with fewer requests outstanding per SM (a compute-free
    // loop with this kernel's loads: 6.59 TB/s at 192 KB in flight per SM, 6.64 at 128 KB, 6.8 at 96 KB).
    // Four warps per CTA still cover the arithmetic (three do not).
    // With a sliding window every row longer than the window attends over exactly the window, so the
    // wave is uniform by construction and shorter splits qualify (rows of 4096: 86.3 -> 82.2 us).
    const int slim_min_tokens = p.window > 0 ? kSlimMinWindowSplitTokens : kSlimMinSplitTokens;
    const bool slim = ctas > sms && ctas <= 2ll * sms && p.split_tokens >= slim_min_tokens;
    return slim ? launch_one_staged<D, WIDE, ROPE, kSlimWarps>(k_map, v_map, p, B, stream)
                : launch_one_staged<D, WIDE, ROPE, kWarps>(k_map, v_map, p, B, stream);
}

}  // namespace

cudaError_t attn_set_attributes(int smem_optin) {
    if (Smem<128, kFatWarps>::TOTAL > smem_optin) return cudaErrorInvalidConfiguration;
    cudaError_t e;
#define AC_SET_STAGED(D_, W_, R_, S_)                                                              \
    e = cudaFuncSetAttribute(paged_decode_attn_kernel<D_, W_, R_, S_>,                             \
                             cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D_, S_>::TOTAL);    \
    if (e != cudaSuccess) return e;                                                                \
    e = cudaFuncSetAttribute(paged_decode_attn_kernel<D_, W_, R_, S_>,                             \
                             cudaFuncAttributeNonPortableClusterSizeAllowed, 1);                   \
    if (e != cudaSuccess) return e;
#define AC_SET_ONE(D_, W_, R_)                                                                    \
    AC_SET_STAGED(D_, W_, R_, kWarps) AC_SET_STAGED(D_, W_, R_, kFatWarps) AC_SET_STAGED(D_, W_, R_, kSlimWarps)
#define AC_SET(D_, W_)                                                                             \
    AC_SET_ONE(D_, W_, ROPE_NONE) AC_SET_ONE(D_, W_, ROPE_PLAIN) AC_SET_ONE(D_, W_, ROPE_VARIANT)
    AC_SET(128, false)
    AC_SET(128, true)
    AC_SET(64, false)
    AC_SET(64, true)
#undef AC_SET_ONE
#undef AC_SET_STAGED
#undef AC_SET
    return cudaSuccess;
}

cudaError_t launch_paged_decode_attn(const CUtensorMap& k_map, const CUtensorMap& v_map,
                                     const void* q_rot,
                                     const int32_t* block_table, int max_pages_per_seq,
                                     const int32_t* context_lens, int new_tokens, float scale,
                                     int num_splits, int split_tokens, float* partial_o,
                                     float* partial_lse, int32_t* arrivals, void* out, int B, int Hq,
                                     int Hkv, int d, int page_size, int32_t* status_flag,
                                     const FusedRopeArgs* rope, int window, const int32_t* row_order,
                                     cudaStream_t stream) {
    AttnParams p;
    p.row_order = row_order;
    p.window = window > 0 ? window : 0;
    p.q_rot_out = nullptr;
    p.k_new = p.v_new = nullptr;
    p.k_cache = p.v_cache = nullptr;
    p.stride_page = p.stride_token = p.stride_head = 0;
    p.rope_cos = p.rope_sin = nullptr;
    p.max_position = p.num_pages = 0;
    p.out_mirror = nullptr;
    if (rope != nullptr) {
        p.out_mirror = static_cast<uint16_t*>(rope->out_mirror);
        p.q_rot_out = static_cast<uint16_t*>(rope->q_rot_out);
        p.k_new = static_cast<const uint16_t*>(rope->k_new);
        p.v_new = static_cast<const uint16_t*>(rope->v_new);
        p.k_cache = static_cast<uint16_t*>(rope->k_cache);
        p.v_cache = static_cast<uint16_t*>(rope->v_cache);
        p.stride_page = rope->stride_page;
        p.stride_token = rope->stride_token;
        p.stride_head = rope->stride_head;
        p.rope_cos = rope->rope_cos;
        p.rope_sin = rope->rope_sin;
        p.max_position = rope->max_position;
        p.num_pages = rope->num_pages;
    }
    p.arrivals = arrivals;
    p.fused_merge = arrivals != nullptr ? 1 : 0;
    // Worth its ~1 us per CTA only when the grid does not fit on the GPU at once, and kept to batch
    // sizes whose ranking (B comparisons per thread) stays short.
    int sms = 0, dev = 0;
    cudaGetDevice(&dev);
    sms = device_state(dev).sm_count;
    p.longest_first = (B > 1 && B <= kLongestFirstMaxBatch &&
                       static_cast<long long>(B) * Hkv * num_splits > 2ll * sms) ? 1 : 0;
    // Merge inside a cluster when the splits of a (request, KV head) fit in one cluster and the grid
    // has no more CTAs than the GPU has SMs.  Clusters are scheduled as a unit inside one GPC: on a
    // fuller GPU some of them wait for a second wave even where the occupancy query says they all
    // fit (32 clusters of 8 CTAs measured 53 us against 35 us with the ticket merge), which costs far
    // more than the merge saves; small grids are where the merge's latency matters anyway.
    p.cluster_merge = (p.fused_merge && num_splits >= 2 && num_splits <= kClusterMergeMaxSplits &&
                       static_cast<long long>(B) * Hkv * num_splits <= sms) ? 1 : 0;
    p.q = static_cast<const uint16_t*>(q_rot);
    p.block_table = block_table;
    p.context_lens = context_lens;
    p.partial_o = partial_o;
    p.partial_lse = partial_lse;
    p.out = static_cast<uint16_t*>(out);
    p.status_flag = status_flag;
    p.scale_log2 = scale * LOG2E;
    p.max_pages_per_seq = max_pages_per_seq;
    p.new_tokens = new_tokens;
    p.num_splits = num_splits;
    p.split_tokens = split_tokens;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.page_size = page_size;
    p.rotary_dim = d;
    p.interleaved = 0;
    p.q_norm_w = p.k_norm_w = nullptr;
    p.norm_eps = 0.0f;
    const bool wide = Hq / Hkv > 8;
    if (rope != nullptr && rope->variant != nullptr) {
        p.rotary_dim = rope->variant->rotary_dim;
        p.interleaved = rope->variant->interleaved;
        p.q_norm_w = static_cast<const uint16_t*>(rope->variant->q_norm_weight);
        p.k_norm_w = static_cast<const uint16_t*>(rope->variant->k_norm_weight);
        p.norm_eps = rope->variant->norm_eps;
        if (d == 128) {
            return wide ? launch_one<128, true, ROPE_VARIANT>(k_map, v_map, p, B, stream)
                        : launch_one<128, false, ROPE_VARIANT>(k_map, v_map, p, B, stream);
        }
        return wide ? launch_one<64, true, ROPE_VARIANT>(k_map, v_map, p, B, stream)
                    : launch_one<64, false, ROPE_VARIANT>(k_map, v_map, p, B, stream);
    }
    if (rope != nullptr) {
        if (d == 128) {
            return wide ? launch_one<128, true, ROPE_PLAIN>(k_map, v_map, p, B, stream)
                        : launch_one<128, false, ROPE_PLAIN>(k_map, v_map, p, B, stream);
        }
        return wide ? launch_one<64, true, ROPE_PLAIN>(k_map, v_map, p, B, stream)
                    : launch_one<64, false, ROPE_PLAIN>(k_map, v_map, p, B, stream);
    }
    if (d == 128) {
        return wide ? launch_one<128, true, ROPE_NONE>(k_map, v_map, p, B, stream)
                    : launch_one<128, false, ROPE_NONE>(k_map, v_map, p, B, stream);
    }
    return wide ? launch_one<64, true, ROPE_NONE>(k_map, v_map, p, B, stream)
                : launch_one<64, false, ROPE_NONE>(k_map, v_map, p, B, stream);
}

}  // namespace ac
