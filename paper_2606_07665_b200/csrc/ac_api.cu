// The C ABI of libac: argument validation, the split plan, tensor-map construction and the launches.
#include <math.h>
#include <stdlib.h>

#include <mutex>

#include "ac_internal.h"

namespace ac {

namespace {

DeviceState g_devices[kMaxDevices];
std::mutex g_init_mutex;                 // ac_init may be called from one host thread per device
thread_local int t_last_cuda_error = 0;
int g_last_sm_count = 0;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode_tiled = nullptr;

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct Shape {
    int B, Hq, Hkv, d, page_size, num_pages;
};

// Largest batch the warp-MMA projection kernels take; beyond it the tcgen05 kernels are used.
constexpr int kWarpMmaMaxBatch = 16;

int check_shape(const Shape& s) {
    if (s.B <= 0 || s.Hq <= 0 || s.Hkv <= 0 || s.d <= 0 || s.page_size <= 0 || s.num_pages <= 0)
        return AC_ERR_SHAPE;
    if (s.Hq % s.Hkv != 0) return AC_ERR_SHAPE;
    if (s.d != 64 && s.d != 128) return AC_ERR_UNSUPPORTED;
    if (s.page_size % 16 != 0 || s.page_size > 256) return AC_ERR_UNSUPPORTED;
    if (s.Hq / s.Hkv > 16) return AC_ERR_UNSUPPORTED;
    if (s.B > 65535 || s.Hq > 65535) return AC_ERR_UNSUPPORTED;
    return AC_OK;
}

int check_strides(const Shape& s, int64_t stride_page, int64_t stride_token, int64_t stride_head) {
    if (stride_page <= 0 || stride_token <= 0 || stride_head <= 0) return AC_ERR_SHAPE;
    if (stride_page % 8 || stride_token % 8 || stride_head % 8) return AC_ERR_ALIGN;
    if (stride_token < s.d || stride_head < s.d) return AC_ERR_SHAPE;
    return AC_OK;
}

int current_ready_device(int* device_out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda(static_cast<int>(e));
    if (dev < 0 || dev >= kMaxDevices || !g_devices[dev].ready) return AC_ERR_NOT_INIT;
    *device_out = dev;
    return AC_OK;
}

// 5-D view of one cache pool for box loads of 16 tokens x head_dim of one head:
// (64 elements, token-in-page, 64-element block of head_dim, head, page).  The block dimension has a
// 128-byte stride, smaller than the token stride before it: tensor-map strides need not be ordered.
int make_cache_map(CUtensorMap* map, const void* base, const Shape& s, int64_t stride_page,
                   int64_t stride_token, int64_t stride_head) {
    cuuint64_t dims[5] = {64, static_cast<cuuint64_t>(s.page_size), static_cast<cuuint64_t>(s.d / 64),
                          static_cast<cuuint64_t>(s.Hkv), static_cast<cuuint64_t>(s.num_pages)};
    cuuint64_t strides[4] = {static_cast<cuuint64_t>(stride_token) * 2, 128,
                             static_cast<cuuint64_t>(stride_head) * 2,
                             static_cast<cuuint64_t>(stride_page) * 2};
    cuuint32_t box[5] = {64, 16, static_cast<cuuint32_t>(s.d / 64), 1, 1};
    cuuint32_t elem_strides[5] = {1, 1, 1, 1, 1};
    CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims,
                                strides, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail_cuda(static_cast<int>(r));
    return AC_OK;
}

}  // namespace

DeviceState& device_state(int device) { return g_devices[device]; }

int fail_cuda(int code) {
    t_last_cuda_error = code;
    return AC_ERR_CUDA;
}

int split_tokens_for(int max_context_len, int num_splits) {
    if (max_context_len < 1) max_context_len = 1;
    if (num_splits < 1) num_splits = 1;
    const long long per = (static_cast<long long>(max_context_len) + num_splits - 1) / num_splits;
    const long long rounded = (per + 63) / 64 * 64;
    return static_cast<int>(rounded > 0x7fffffc0ll ? 0x7fffffc0ll : rounded);
}

}  // namespace ac

using namespace ac;

extern "C" {

int ac_init(int device) {
    cudaError_t e;
    if (device < 0) {
        e = cudaGetDevice(&device);
        if (e != cudaSuccess) return fail_cuda(static_cast<int>(e));
    }
    if (device >= kMaxDevices) return AC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_init_mutex);
    int prev = -1;
    e = cudaGetDevice(&prev);
    if (e != cudaSuccess) return fail_cuda(static_cast<int>(e));
    if (prev != device) {
        e = cudaSetDevice(device);
        if (e != cudaSuccess) return fail_cuda(static_cast<int>(e));
    }
    int status = AC_OK;
    DeviceState st;
    int major = 0;
    do {
        if ((e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, device)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&st.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device)) != cudaSuccess) {
            status = fail_cuda(static_cast<int>(e));
            break;
        }
        if (major != 10) {          // the kernels are built for sm_100a only
            status = AC_ERR_UNSUPPORTED;
            break;
        }
        if (g_encode_tiled == nullptr) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
            if (e != cudaSuccess || fn == nullptr || qres != cudaDriverEntryPointSuccess) {
                status = fail_cuda(static_cast<int>(e != cudaSuccess ? e : cudaErrorSymbolNotFound));
                break;
            }
            g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
        }
        e = attn_set_attributes(st.smem_optin);
        if (e == cudaSuccess) e = qkv_set_attributes(st.smem_optin);
        if (e == cudaSuccess) e = proj_tc_set_attributes(st.smem_optin);
        if (e != cudaSuccess) {
            status = fail_cuda(static_cast<int>(e));
            break;
        }
        st.ready = true;
        g_devices[device] = st;
        g_last_sm_count = st.sm_count;
    } while (false);
    if (prev != device) cudaSetDevice(prev);
    return status;
}

const char* ac_status_string(int status) {
    switch (status) {
        case AC_OK: return "ok";
        case AC_ERR_NULL: return "a required pointer is NULL";
        case AC_ERR_SHAPE: return "a size or stride is non-positive or inconsistent";
        case AC_ERR_UNSUPPORTED: return "shape, layout or device outside the supported set";
        case AC_ERR_ALIGN: return "pointer or stride not aligned to 16 bytes";
        case AC_ERR_WORKSPACE: return "workspace missing or too small for num_splits";
        case AC_ERR_CUDA: return "a CUDA call failed (see ac_last_cuda_error)";
        case AC_ERR_NOT_INIT: return "ac_init has not succeeded on the current device";
        case AC_ERR_SCRATCH_LIMIT:
            return "partials for this B, Hq, d, num_splits exceed the library's built-in scratch "
                   "(AC_STATIC_SCRATCH_BYTES); use fewer splits or ac_paged_decode_attn with a workspace";
        default: return "unknown status";
    }
}

int ac_last_cuda_error(void) { return t_last_cuda_error; }

int ac_sm_count(void) { return g_last_sm_count; }

int ac_split_tokens(int max_context_len, int num_splits) {
    return split_tokens_for(max_context_len, num_splits);
}

size_t ac_workspace_bytes(int B, int Hq, int d, int num_splits) {
    if (B <= 0 || Hq <= 0 || d <= 0 || num_splits <= 1) return 0;
    return static_cast<size_t>(B) * Hq * num_splits * (static_cast<size_t>(d) + 1) * sizeof(float);
}

// The plan proper.  token_counts == nullptr: every row is taken to attend over max_context_len
// tokens; otherwise token_counts[b] = tokens row b attends over (<= 0: the row launches no work).
// How many thread-block clusters of `size` one-per-SM CTAs are resident at once.  A cluster lives inside
// one GPC, so this is well below sm_count / size for the larger sizes.  For the 148-SM part the figures
// are what cudaOccupancyMaxActiveClusters reports for the twelve-warp attention kernel (the launch asks
// the runtime itself and falls back to the ticket merge when a grid has more clusters than that; the
// plan only needs to know it in advance to price the merge correctly); other parts get a cautious
// guess.
static int cluster_capacity(int size, int sm_count) {
    static const int b200[17] = {0, 148, 74, 45, 33, 26, 22, 15, 15, 15, 11, 7, 7, 7, 7, 7, 7};
    if (size < 1 || size > 16) return 0;
    if (sm_count == 148) return b200[size];
    return (sm_count / size) * 3 / 4;
}

static int plan_splits(int B, int Hq, int Hkv, int d, int page_size, int max_context_len, int sm_count,
                       const int32_t* token_counts, int* num_splits_out, int* split_tokens_out,
                       size_t* workspace_bytes_out) {
    if (num_splits_out == nullptr || split_tokens_out == nullptr || workspace_bytes_out == nullptr)
        return AC_ERR_NULL;
    Shape s{B, Hq, Hkv, d, page_size, 1};
    int st = check_shape(s);
    if (st != AC_OK) return st;
    if (max_context_len <= 0) return AC_ERR_SHAPE;
    if (sm_count <= 0) sm_count = g_last_sm_count > 0 ? g_last_sm_count : 148;

    // Two CTAs are resident per SM ("slots").  Measured on B200: one CTA on its own streams ~45-57
    // GB/s once its ring is full (96 KB in flight against ~2 us of load latency); charged with its
    // own ramp that is ~33 GB/s over a short chunk, the figure fitted to sweeps of the split count.
    // A wave of CTAs costs ~3 us of ramp-up/epilogue that overlaps poorly, and every extra split adds
    // partial-result traffic.
    //  * At least one wave of (request, KV head) pairs: do not split, unless contexts are long --
    //    then cut them into chunks of at most 4096 tokens so that ragged batches balance.
    //  * Fewer pairs than slots: scan the split counts and take the one with the smallest
    //    estimated time.  Without the rows' lengths every row counts as max_context_len tokens; with
    //    them, a split that lies beyond a row's end costs nothing (its CTA exits at once), so a ragged
    //    batch can take more, shorter splits before it spills into a second wave.
    const double slots = 2.0 * sm_count;
    const double hbm = 6.5e12 * sm_count / 148.0;      // bytes/s the whole GPU streams
    const double cta_rate = 33e9;                       // bytes/s one CTA streams on its own
    // Grids of at most one CTA per SM with splits longer than 192 tokens run twelve warps per CTA
    // (launch_one in paged_decode_attn.cu); fitted to sweeps of the split count like the figure above.
    const double fat_cta_rate = 75e9;
    const double wave_cost = 3e-6;
    // A grid that could have fitted the GPU at once but spills into a further wave pays much more than
    // a ramp for it: the CTAs of that wave start only when first-wave CTAs retire and then need their
    // whole own duration (measured on batches of 32 requests: 295 CTAs 19 us, 350 CTAs 30 us; 256 CTAs
    // 34 us, 415 CTAs 43 us).
    const double spill_wave_cost = 8e-6;
    long long active_rows = B;
    double total_tokens = static_cast<double>(B) * max_context_len;
    if (token_counts != nullptr) {
        active_rows = 0;
        total_tokens = 0.0;
        for (int b = 0; b < B; ++b)
            if (token_counts[b] > 0) {
                ++active_rows;
                total_tokens += token_counts[b] < max_context_len ? token_counts[b] : max_context_len;
            }
        if (active_rows == 0) active_rows = 1;
    }
    const long long pairs = active_rows * Hkv;
    long long S = 1;
    if (pairs >= static_cast<long long>(slots)) {
        S = (static_cast<long long>(max_context_len) + 4095) / 4096;
    } else {
        // Splits are at least 256 tokens long -- 128 where the merge is the cheap one inside a cluster
        // (small grids, where nothing but latency is at stake).
        int s_max = (max_context_len + 63) / 64;            // the chunk-length test below does the limiting
        if (s_max > 4096) s_max = 4096;
        if (token_counts != nullptr && static_cast<long long>(s_max) * B > 4000000ll) {
            s_max = static_cast<int>(4000000ll / B);      // bound the host work of the scan
            if (s_max < 1) s_max = 1;
        }
        double best = 0.0;
        for (int cand = 1; cand <= s_max; ++cand) {
            const int chunk = split_tokens_for(max_context_len, cand);
            if (static_cast<long long>(chunk) * (cand - 1) >= max_context_len) continue;   // empty split
            // the launch decides by the grid it is given: all B rows count, active or not
            const bool in_cluster = cand <= kClusterMergeMaxSplits &&
                                    static_cast<long long>(B) * Hkv * cand <= sm_count &&
                                    static_cast<long long>(B) * Hkv <= cluster_capacity(cand, sm_count);
            if (cand > 1 && chunk < (in_cluster ? 128 : 256)) continue;
            const bool fat = static_cast<long long>(B) * Hkv * cand <= sm_count && chunk > 192;
            const double rate = fat ? fat_cta_rate : cta_rate;
            double n = static_cast<double>(pairs) * cand;                // CTAs that have tokens
            double longest = chunk;                                       // tokens of the longest CTA
            if (token_counts != nullptr) {
                long long pieces = 0;
                int most = 0;
                for (int b = 0; b < B; ++b) {
                    int t = token_counts[b];
                    if (t <= 0) continue;
                    if (t > max_context_len) t = max_context_len;
                    pieces += (t + chunk - 1) / chunk;
                    const int m = t < chunk ? t : chunk;
                    if (m > most) most = m;
                }
                n = static_cast<double>(pieces) * Hkv;
                longest = most;
            }
            const double bytes_per_token = d * 4.0;                      // K + V of one KV head
            const double waves = ceil(n / slots);
            double t;
            if (token_counts == nullptr) {
                const double c = longest * bytes_per_token;
                const double last = n - (waves - 1.0) * slots;
                t = (waves - 1.0) * slots * c / hbm;
                const double t_last_bw = last * c / hbm, t_last_cta = c / rate;
                t += (t_last_bw > t_last_cta ? t_last_bw : t_last_cta) + wave_cost + (waves - 1.0) * spill_wave_cost;
            } else {
                const double t_bw = total_tokens * Hkv * bytes_per_token / hbm;
                const double t_cta = longest * bytes_per_token / rate;
                t = (t_bw > t_cta ? t_bw : t_cta) + wave_cost + (waves - 1.0) * spill_wave_cost;
            }
            if (cand > 1)            // partials out and back in plus the ticket round trip, or two cluster barriers
                t += in_cluster ? 0.3e-6 : 2.0 * active_rows * Hq * cand * (d + 1.0) * 4.0 / hbm + 1.6e-6;
            if (best == 0.0 || t < best) {
                best = t;
                S = cand;
            }
        }
    }
    if (pairs < static_cast<long long>(slots) && pairs * S <= static_cast<long long>(slots) &&
        split_tokens_for(max_context_len, static_cast<int>(S)) >= 8192) {
        // Very long contexts in a single wave.  The launch runs such grids with four warps per CTA
        // (launch_one in paged_decode_attn.cu: splits of at least 8192 tokens, more than one and at most
        // two CTAs per SM), which streams fastest when the wave is full: take the most splits that still
        // fit the slots and stay that long (long-context workload: 309 us; six-warp CTAs in one wave 326-330 us,
        // in 1.75 waves of shorter chunks 315 us).
        long long full = static_cast<long long>(slots) / pairs;
        while (full > S && split_tokens_for(max_context_len, static_cast<int>(full)) < 8192) --full;
        if (full > S) S = full;
    }
    if (S < 1) S = 1;
    if (S > 65535) S = 65535;
    int chunk = split_tokens_for(max_context_len, static_cast<int>(S));
    // Drop splits that the rounding of the chunk length made empty for every row.
    S = (static_cast<long long>(max_context_len) + chunk - 1) / chunk;
    *num_splits_out = static_cast<int>(S);
    *split_tokens_out = split_tokens_for(max_context_len, static_cast<int>(S));
    *workspace_bytes_out = ac_workspace_bytes(B, Hq, d, static_cast<int>(S));
    return AC_OK;
}

int ac_decode_plan(int B, int Hq, int Hkv, int d, int page_size, int max_context_len, int sm_count,
                   int* num_splits_out, int* split_tokens_out, size_t* workspace_bytes_out) {
    return plan_splits(B, Hq, Hkv, d, page_size, max_context_len, sm_count, nullptr, num_splits_out,
                       split_tokens_out, workspace_bytes_out);
}

int ac_decode_plan_for_lengths(const int32_t* token_counts_host, int B, int Hq, int Hkv, int d,
                               int page_size, int max_context_len, int sm_count, int* num_splits_out,
                               int* split_tokens_out, size_t* workspace_bytes_out) {
    if (token_counts_host == nullptr) return AC_ERR_NULL;
    return plan_splits(B, Hq, Hkv, d, page_size, max_context_len, sm_count, token_counts_host,
                       num_splits_out, split_tokens_out, workspace_bytes_out);
}

// Checks ac_rope_options and translates them; *out stays nullptr when they describe the plain rotation.
static int parse_rope_options(const ac_rope_options* options, int d, RopeVariant* variant,
                              const RopeVariant** out) {
    *out = nullptr;
    if (options == nullptr) return AC_OK;
    const int rd = options->rotary_dim == 0 ? d : options->rotary_dim;
    if (rd < 2 || rd > d || (rd & 1)) return AC_ERR_SHAPE;
    const bool plain = rd == d && !options->interleaved && !options->q_norm_weight && !options->k_norm_weight;
    if (plain) return AC_OK;
    variant->rotary_dim = rd;
    variant->interleaved = options->interleaved ? 1 : 0;
    variant->q_norm_weight = options->q_norm_weight;
    variant->k_norm_weight = options->k_norm_weight;
    variant->norm_eps = options->norm_eps;
    if ((variant->q_norm_weight || variant->k_norm_weight) && !(options->norm_eps >= 0.0f)) return AC_ERR_SHAPE;
    if ((variant->q_norm_weight && !aligned16(variant->q_norm_weight)) ||
        (variant->k_norm_weight && !aligned16(variant->k_norm_weight)))
        return AC_ERR_ALIGN;
    *out = variant;
    return AC_OK;
}

int ac_rope_kv_append_ex(const void* q_in, void* q_out, const void* k_new, const void* v_new,
                         void* k_cache, void* v_cache, int64_t stride_page, int64_t stride_token,
                         int64_t stride_head, const int32_t* block_table, int max_pages_per_seq,
                         const int32_t* context_lens, const float* rope_cos, const float* rope_sin,
                         int max_position, int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                         int32_t* status_flag, void* stream, const ac_rope_options* options) {
    if (!q_in || !q_out || !k_new || !v_new || !k_cache || !v_cache || !block_table || !context_lens ||
        !rope_cos || !rope_sin)
        return AC_ERR_NULL;
    Shape s{B, Hq, Hkv, d, page_size, num_pages};
    int st = check_shape(s);
    if (st != AC_OK) return st;
    if (max_pages_per_seq <= 0 || max_position <= 0) return AC_ERR_SHAPE;
    st = check_strides(s, stride_page, stride_token, stride_head);
    if (st != AC_OK) return st;
    if (!aligned16(q_in) || !aligned16(q_out) || !aligned16(k_new) || !aligned16(v_new) ||
        !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(rope_cos) || !aligned16(rope_sin))
        return AC_ERR_ALIGN;
    RopeVariant variant;
    const RopeVariant* vp = nullptr;
    st = parse_rope_options(options, d, &variant, &vp);
    if (st != AC_OK) return st;
    int dev;
    st = current_ready_device(&dev);
    if (st != AC_OK) return st;
    cudaError_t e = launch_rope_kv_append(q_in, q_out, k_new, v_new, k_cache, v_cache, stride_page,
                                          stride_token, stride_head, block_table, max_pages_per_seq,
                                          context_lens, rope_cos, rope_sin, max_position, B, Hq, Hkv, d,
                                          page_size, num_pages, status_flag, vp,
                                          static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AC_OK : fail_cuda(static_cast<int>(e));
}

int ac_rope_kv_append(const void* q_in, void* q_out, const void* k_new, const void* v_new,
                      void* k_cache, void* v_cache, int64_t stride_page, int64_t stride_token,
                      int64_t stride_head, const int32_t* block_table, int max_pages_per_seq,
                      const int32_t* context_lens, const float* rope_cos, const float* rope_sin,
                      int max_position, int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                      int32_t* status_flag, void* stream) {
    return ac_rope_kv_append_ex(q_in, q_out, k_new, v_new, k_cache, v_cache, stride_page, stride_token,
                                stride_head, block_table, max_pages_per_seq, context_lens, rope_cos,
                                rope_sin, max_position, B, Hq, Hkv, d, page_size, num_pages, status_flag,
                                stream, nullptr);
}

int ac_qkv_rope_kv_append(const void* x, const void* w_qkv, int H, void* q_out, void* k_cache,
                          void* v_cache, int64_t stride_page, int64_t stride_token, int64_t stride_head,
                          const int32_t* block_table, int max_pages_per_seq,
                          const int32_t* context_lens, const float* rope_cos, const float* rope_sin,
                          int max_position, int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                          int32_t* status_flag, void* stream) {
    return ac_qkv_rope_kv_append_ex(x, w_qkv, H, q_out, k_cache, v_cache, stride_page, stride_token,
                                    stride_head, block_table, max_pages_per_seq, context_lens, rope_cos,
                                    rope_sin, max_position, B, Hq, Hkv, d, page_size, num_pages, status_flag,
                                    stream, nullptr);
}

int ac_qkv_rope_kv_append_ex(const void* x, const void* w_qkv, int H, void* q_out, void* k_cache,
                             void* v_cache, int64_t stride_page, int64_t stride_token, int64_t stride_head,
                             const int32_t* block_table, int max_pages_per_seq,
                             const int32_t* context_lens, const float* rope_cos, const float* rope_sin,
                             int max_position, int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                             int32_t* status_flag, void* stream, const ac_rope_options* options) {
    if (!x || !w_qkv || !q_out || !k_cache || !v_cache || !block_table || !context_lens || !rope_cos ||
        !rope_sin)
        return AC_ERR_NULL;
    Shape s{B, Hq, Hkv, d, page_size, num_pages};
    int st = check_shape(s);
    if (st != AC_OK) return st;
    if (H <= 0 || max_pages_per_seq <= 0 || max_position <= 0) return AC_ERR_SHAPE;
    if (H % 64 != 0) return AC_ERR_UNSUPPORTED;
    st = check_strides(s, stride_page, stride_token, stride_head);
    if (st != AC_OK) return st;
    if (!aligned16(x) || !aligned16(w_qkv) || !aligned16(q_out) || !aligned16(k_cache) ||
        !aligned16(v_cache))
        return AC_ERR_ALIGN;
    RopeVariant variant;
    const RopeVariant* vp = nullptr;
    st = parse_rope_options(options, d, &variant, &vp);
    if (st != AC_OK) return st;
    int dev;
    st = current_ready_device(&dev);
    if (st != AC_OK) return st;

    // W [(Hq+2Hkv)*d, H] as (64 elements, row inside a half head, half, head, 64-element K block);
    // x [B, H] as (64 elements, batch row, 64-element K block).
    const cuuint64_t row_bytes = static_cast<cuuint64_t>(H) * 2;
    CUtensorMap w_map, x_map;
    if (B > kWarpMmaMaxBatch) {
        // Batched decode: batch tiles of up to 128 rows on the tcgen05 path (boxes of 24 pairs x 2 K blocks).
        cuuint64_t wdims[5] = {64, static_cast<cuuint64_t>(d / 2), 2, static_cast<cuuint64_t>(Hq + 2 * Hkv),
                               static_cast<cuuint64_t>(H / 64)};
        cuuint64_t wstrides[4] = {row_bytes, row_bytes * (d / 2), row_bytes * d, 128};
        // 24 pairs per tile (plain epilogue: overlapping tiles), 32 with the prelude variants (disjoint tiles)
        cuuint32_t wbox[5] = {64, static_cast<cuuint32_t>(vp != nullptr ? 32 : 24), 2, 1,
                              static_cast<cuuint32_t>(proj_tc_k_blocks(B))};
        cuuint32_t es5[5] = {1, 1, 1, 1, 1};
        CUresult r = g_encode_tiled(&w_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(w_qkv),
                                    wdims, wstrides, wbox, es5, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail_cuda(static_cast<int>(r));
        cuuint64_t xdims[3] = {64, static_cast<cuuint64_t>(B), static_cast<cuuint64_t>(H / 64)};
        cuuint64_t xstrides[2] = {row_bytes, 128};
        cuuint32_t xbox[3] = {64, static_cast<cuuint32_t>(proj_tc_batch_rows(B)), static_cast<cuuint32_t>(proj_tc_k_blocks(B))};
        cuuint32_t es3[3] = {1, 1, 1};
        r = g_encode_tiled(&x_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), xdims, xstrides,
                           xbox, es3, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail_cuda(static_cast<int>(r));
        cudaError_t e = launch_qkv_rope_kv_append_tc(w_map, x_map, q_out, k_cache, v_cache, stride_page,
                                                     stride_token, stride_head, block_table,
                                                     max_pages_per_seq, context_lens, rope_cos, rope_sin,
                                                     max_position, B, H, Hq, Hkv, d, page_size, num_pages,
                                                     status_flag, vp, static_cast<cudaStream_t>(stream));
        return e == cudaSuccess ? AC_OK : fail_cuda(static_cast<int>(e));
    }
    {
        cuuint64_t dims[5] = {64, static_cast<cuuint64_t>(d / 2), 2, static_cast<cuuint64_t>(Hq + 2 * Hkv),
                              static_cast<cuuint64_t>(H / 64)};
        cuuint64_t strides[4] = {row_bytes, row_bytes * (d / 2), row_bytes * d, 128};
        cuuint32_t box[5] = {64, 16, 2, 1, 4};
        cuuint32_t es[5] = {1, 1, 1, 1, 1};
        CUresult r = g_encode_tiled(&w_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(w_qkv),
                                    dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail_cuda(static_cast<int>(r));
    }
    {
        cuuint64_t dims[3] = {64, static_cast<cuuint64_t>(B), static_cast<cuuint64_t>(H / 64)};
        cuuint64_t strides[2] = {row_bytes, 128};
        cuuint32_t box[3] = {64, static_cast<cuuint32_t>(qkv_batch_tile(B)), 4};
        cuuint32_t es[3] = {1, 1, 1};
        CUresult r = g_encode_tiled(&x_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims,
                                    strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail_cuda(static_cast<int>(r));
    }
    cudaError_t e = launch_qkv_rope_kv_append(w_map, x_map, q_out, k_cache, v_cache, stride_page,
                                              stride_token, stride_head, block_table, max_pages_per_seq,
                                              context_lens, rope_cos, rope_sin, max_position, B, H, Hq,
                                              Hkv, d, page_size, num_pages, status_flag, vp,
                                              static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AC_OK : fail_cuda(static_cast<int>(e));
}

int ac_oproj_residual_rmsnorm(const void* attn_out, const void* w_o, int K, int N,
                              const void* residual_in, void* residual_out, const void* norm_weight,
                              float norm_eps, void* normed_out, int B, void* stream) {
    if (!attn_out || !w_o || !residual_in || !residual_out || !norm_weight || !normed_out) return AC_ERR_NULL;
    if (B <= 0 || K <= 0 || N <= 0 || !(norm_eps >= 0.0f)) return AC_ERR_SHAPE;
    if (K % 64 != 0 || N % 32 != 0 || B > 65535) return AC_ERR_UNSUPPORTED;
    if (!aligned16(attn_out) || !aligned16(w_o) || !aligned16(residual_in) || !aligned16(residual_out) ||
        !aligned16(norm_weight) || !aligned16(normed_out))
        return AC_ERR_ALIGN;
    int dev;
    int st = current_ready_device(&dev);
    if (st != AC_OK) return st;
    // W_o [N, K] as (64 elements, row inside a 16-row block, -, 16-row block, 64-element K block);
    // attn_out [B, K] as (64 elements, batch row, 64-element K block).
    const cuuint64_t row_bytes = static_cast<cuuint64_t>(K) * 2;
    CUtensorMap w_map, x_map;
    cudaStream_t cs_tc = static_cast<cudaStream_t>(stream);
    if (B > kWarpMmaMaxBatch) {
        cuuint64_t wdims[5] = {64, 16, 2, static_cast<cuuint64_t>(N / 32), static_cast<cuuint64_t>(K / 64)};
        cuuint64_t wstrides[4] = {row_bytes, row_bytes * 16, row_bytes * 32, 128};
        cuuint32_t wbox[5] = {64, 16, 2, 1, static_cast<cuuint32_t>(proj_tc_k_blocks(B))};
        cuuint32_t es5[5] = {1, 1, 1, 1, 1};
        CUresult r = g_encode_tiled(&w_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(w_o), wdims,
                                    wstrides, wbox, es5, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail_cuda(static_cast<int>(r));
        cuuint64_t xdims[3] = {64, static_cast<cuuint64_t>(B), static_cast<cuuint64_t>(K / 64)};
        cuuint64_t xstrides[2] = {row_bytes, 128};
        cuuint32_t xbox[3] = {64, static_cast<cuuint32_t>(proj_tc_batch_rows(B)), static_cast<cuuint32_t>(proj_tc_k_blocks(B))};
        cuuint32_t es3[3] = {1, 1, 1};
        r = g_encode_tiled(&x_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(attn_out), xdims,
                           xstrides, xbox, es3, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail_cuda(static_cast<int>(r));
        cudaError_t e = launch_oproj_residual_tc(w_map, x_map, residual_in, residual_out, B, K, N, cs_tc);
        if (e != cudaSuccess) return fail_cuda(static_cast<int>(e));
        e = launch_rmsnorm_rows(residual_out, norm_weight, normed_out, B, N, norm_eps, cs_tc);
        return e == cudaSuccess ? AC_OK : fail_cuda(static_cast<int>(e));
    }
    {
        // 16 consecutive rows per CTA (the third dimension is a dummy of extent 1)
        cuuint64_t dims[5] = {64, 16, 1, static_cast<cuuint64_t>(N / 16), static_cast<cuuint64_t>(K / 64)};
        cuuint64_t strides[4] = {row_bytes, row_bytes * 16, row_bytes * 16, 128};
        cuuint32_t box[5] = {64, 16, 1, 1, 4};
        cuuint32_t es[5] = {1, 1, 1, 1, 1};
        CUresult r = g_encode_tiled(&w_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(w_o), dims,
                                    strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail_cuda(static_cast<int>(r));
    }
    {
        cuuint64_t dims[3] = {64, static_cast<cuuint64_t>(B), static_cast<cuuint64_t>(K / 64)};
        cuuint64_t strides[2] = {row_bytes, 128};
        cuuint32_t box[3] = {64, static_cast<cuuint32_t>(qkv_batch_tile(B)), 4};
        cuuint32_t es[3] = {1, 1, 1};
        CUresult r = g_encode_tiled(&x_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(attn_out),
                                    dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail_cuda(static_cast<int>(r));
    }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    cudaError_t e = launch_oproj_residual(w_map, x_map, residual_in, residual_out, B, K, N, cs);
    if (e != cudaSuccess) return fail_cuda(static_cast<int>(e));
    e = launch_rmsnorm_rows(residual_out, norm_weight, normed_out, B, N, norm_eps, cs);
    return e == cudaSuccess ? AC_OK : fail_cuda(static_cast<int>(e));
}

static int attn_common(const void* q_rot, const void* k_cache, const void* v_cache, int64_t stride_page,
                       int64_t stride_token, int64_t stride_head, const int32_t* block_table,
                       int max_pages_per_seq, const int32_t* context_lens, int new_tokens,
                       float softmax_scale, int num_splits, void* workspace, size_t workspace_bytes,
                       void* out, int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                       int max_context_len, int32_t* status_flag, void* stream, bool fused_merge,
                       const FusedRopeArgs* rope = nullptr, int window = 0,
                       const int32_t* row_order = nullptr) {
    if (!q_rot || !k_cache || !v_cache || !block_table || !context_lens) return AC_ERR_NULL;
    Shape s{B, Hq, Hkv, d, page_size, num_pages};
    int st = check_shape(s);
    if (st != AC_OK) return st;
    if (max_pages_per_seq <= 0 || max_context_len <= 0 || num_splits <= 0) return AC_ERR_SHAPE;
    if (new_tokens != 0 && new_tokens != 1) return AC_ERR_UNSUPPORTED;
    if (num_splits > 65535) return AC_ERR_UNSUPPORTED;
    st = check_strides(s, stride_page, stride_token, stride_head);
    if (st != AC_OK) return st;
    if (!aligned16(q_rot) || !aligned16(k_cache) || !aligned16(v_cache)) return AC_ERR_ALIGN;
    float* partial_o = nullptr;
    float* partial_lse = nullptr;
    int32_t* arrivals = nullptr;
    if (num_splits == 1 || fused_merge) {
        if (!out) return AC_ERR_NULL;
        if (!aligned16(out)) return AC_ERR_ALIGN;
    }
    if (num_splits > 1) {
        const size_t need = fused_merge ? ac_fused_workspace_bytes(B, Hq, Hkv, d, num_splits)
                                        : ac_workspace_bytes(B, Hq, d, num_splits);
        if (!workspace || workspace_bytes < need) return AC_ERR_WORKSPACE;
        if (!aligned16(workspace)) return AC_ERR_ALIGN;
        partial_o = static_cast<float*>(workspace);
        partial_lse = partial_o + static_cast<size_t>(B) * Hq * num_splits * d;
        if (fused_merge)
            arrivals = reinterpret_cast<int32_t*>(partial_lse + static_cast<size_t>(B) * Hq * num_splits);
    }
    int dev;
    st = current_ready_device(&dev);
    if (st != AC_OK) return st;
    CUtensorMap k_map, v_map;
    st = make_cache_map(&k_map, k_cache, s, stride_page, stride_token, stride_head);
    if (st != AC_OK) return st;
    st = make_cache_map(&v_map, v_cache, s, stride_page, stride_token, stride_head);
    if (st != AC_OK) return st;
    const float scale = softmax_scale > 0.0f ? softmax_scale : 1.0f / sqrtf(static_cast<float>(d));
    // With a sliding window a row attends over at most window + 63 tokens (its range starts at a
    // multiple of 64 at or below the window's first token).
    if (window < 0) return AC_ERR_SHAPE;
    const int span = (window > 0 && window + 63 < max_context_len) ? window + 63 : max_context_len;
    const int split_tokens = split_tokens_for(span, num_splits);
    cudaError_t e = launch_paged_decode_attn(k_map, v_map, q_rot, block_table,
                                             max_pages_per_seq, context_lens, new_tokens, scale,
                                             num_splits, split_tokens, partial_o, partial_lse, arrivals,
                                             out, B, Hq, Hkv, d, page_size, status_flag, rope, window,
                                             row_order, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AC_OK : fail_cuda(static_cast<int>(e));
}

size_t ac_fused_workspace_bytes(int B, int Hq, int Hkv, int d, int num_splits) {
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || d <= 0 || num_splits <= 1) return 0;
    return ac_workspace_bytes(B, Hq, d, num_splits) + static_cast<size_t>(B) * Hkv * sizeof(int32_t);
}

int ac_fused_workspace_reset(void* workspace, size_t workspace_bytes, int B, int Hq, int Hkv, int d,
                             int num_splits, void* stream) {
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || d <= 0 || num_splits <= 0) return AC_ERR_SHAPE;
    if (num_splits == 1) return AC_OK;                       // nothing to reset
    if (!workspace || workspace_bytes < ac_fused_workspace_bytes(B, Hq, Hkv, d, num_splits))
        return AC_ERR_WORKSPACE;
    char* counters = static_cast<char*>(workspace) + ac_workspace_bytes(B, Hq, d, num_splits);
    cudaError_t e = cudaMemsetAsync(counters, 0, static_cast<size_t>(B) * Hkv * sizeof(int32_t),
                                    static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AC_OK : fail_cuda(static_cast<int>(e));
}

int ac_paged_decode_attn(const void* q_rot, const void* k_cache, const void* v_cache,
                         int64_t stride_page, int64_t stride_token, int64_t stride_head,
                         const int32_t* block_table, int max_pages_per_seq,
                         const int32_t* context_lens, int new_tokens, float softmax_scale,
                         int num_splits, void* workspace, size_t workspace_bytes, void* out, int B,
                         int Hq, int Hkv, int d, int page_size, int num_pages, int max_context_len,
                         int32_t* status_flag, void* stream) {
    return attn_common(q_rot, k_cache, v_cache, stride_page, stride_token, stride_head, block_table,
                       max_pages_per_seq, context_lens, new_tokens, softmax_scale, num_splits, workspace,
                       workspace_bytes, out, B, Hq, Hkv, d, page_size, num_pages, max_context_len,
                       status_flag, stream, false);
}

int ac_paged_decode_attn_fused_merge(const void* q_rot, const void* k_cache, const void* v_cache,
                                     int64_t stride_page, int64_t stride_token, int64_t stride_head,
                                     const int32_t* block_table, int max_pages_per_seq,
                                     const int32_t* context_lens, int new_tokens, float softmax_scale,
                                     int num_splits, void* workspace, size_t workspace_bytes, void* out,
                                     int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                                     int max_context_len, int32_t* status_flag, void* stream) {
    return attn_common(q_rot, k_cache, v_cache, stride_page, stride_token, stride_head, block_table,
                       max_pages_per_seq, context_lens, new_tokens, softmax_scale, num_splits, workspace,
                       workspace_bytes, out, B, Hq, Hkv, d, page_size, num_pages, max_context_len,
                       status_flag, stream, true);
}

int ac_decode_step_fused(const void* q_in, void* q_rot_out, const void* k_new, const void* v_new,
                         void* k_cache, void* v_cache, int64_t stride_page, int64_t stride_token,
                         int64_t stride_head, const int32_t* block_table, int max_pages_per_seq,
                         const int32_t* context_lens, const float* rope_cos, const float* rope_sin,
                         int max_position, float softmax_scale, int num_splits, void* workspace,
                         size_t workspace_bytes, void* out, int B, int Hq, int Hkv, int d, int page_size,
                         int num_pages, int max_context_len, int32_t* status_flag, void* stream) {
    return ac_decode_step_fused_ex(q_in, q_rot_out, k_new, v_new, k_cache, v_cache, stride_page,
                                   stride_token, stride_head, block_table, max_pages_per_seq,
                                   context_lens, rope_cos, rope_sin, max_position, softmax_scale,
                                   num_splits, workspace, workspace_bytes, out, B, Hq, Hkv, d, page_size,
                                   num_pages, max_context_len, status_flag, stream, nullptr);
}

// The fused step with an optional mirror of the result (a second destination for every store to out).
static int decode_step_fused_impl(const void* q_in, void* q_rot_out, const void* k_new, const void* v_new,
                                  void* k_cache, void* v_cache, int64_t stride_page, int64_t stride_token,
                                  int64_t stride_head, const int32_t* block_table, int max_pages_per_seq,
                                  const int32_t* context_lens, const float* rope_cos, const float* rope_sin,
                                  int max_position, float softmax_scale, int num_splits, void* workspace,
                                  size_t workspace_bytes, void* out, int B, int Hq, int Hkv, int d,
                                  int page_size, int num_pages, int max_context_len, int32_t* status_flag,
                                  void* stream, const ac_attn_options* options, void* out_mirror) {
    const int window = options != nullptr ? options->window : 0;
    const int32_t* row_order = options != nullptr ? options->row_order : nullptr;
    if (!q_in || !k_new || !v_new || !rope_cos || !rope_sin) return AC_ERR_NULL;
    if (max_position <= 0) return AC_ERR_SHAPE;
    if (q_rot_out == q_in) return AC_ERR_UNSUPPORTED;      // other CTAs still read the raw rows
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(rope_cos) || !aligned16(rope_sin) ||
        (q_rot_out && !aligned16(q_rot_out)))
        return AC_ERR_ALIGN;
    RopeVariant variant;
    const RopeVariant* vp = nullptr;
    const int pst = parse_rope_options(options != nullptr ? options->rope : nullptr, d, &variant, &vp);
    if (pst != AC_OK) return pst;
    FusedRopeArgs rope;
    rope.variant = vp;
    rope.q_rot_out = q_rot_out;
    rope.k_new = k_new;
    rope.v_new = v_new;
    rope.k_cache = k_cache;
    rope.v_cache = v_cache;
    rope.stride_page = stride_page;
    rope.stride_token = stride_token;
    rope.stride_head = stride_head;
    rope.rope_cos = rope_cos;
    rope.rope_sin = rope_sin;
    rope.max_position = max_position;
    rope.num_pages = num_pages;
    rope.out_mirror = out_mirror;
    return attn_common(q_in, k_cache, v_cache, stride_page, stride_token, stride_head, block_table,
                       max_pages_per_seq, context_lens, 1, softmax_scale, num_splits, workspace,
                       workspace_bytes, out, B, Hq, Hkv, d, page_size, num_pages, max_context_len,
                       status_flag, stream, true, &rope, window, row_order);
}

int ac_decode_step_fused_ex(const void* q_in, void* q_rot_out, const void* k_new, const void* v_new,
                            void* k_cache, void* v_cache, int64_t stride_page, int64_t stride_token,
                            int64_t stride_head, const int32_t* block_table, int max_pages_per_seq,
                            const int32_t* context_lens, const float* rope_cos, const float* rope_sin,
                            int max_position, float softmax_scale, int num_splits, void* workspace,
                            size_t workspace_bytes, void* out, int B, int Hq, int Hkv, int d,
                            int page_size, int num_pages, int max_context_len, int32_t* status_flag,
                            void* stream, const ac_attn_options* options) {
    return decode_step_fused_impl(q_in, q_rot_out, k_new, v_new, k_cache, v_cache, stride_page, stride_token,
                                  stride_head, block_table, max_pages_per_seq, context_lens, rope_cos,
                                  rope_sin, max_position, softmax_scale, num_splits, workspace,
                                  workspace_bytes, out, B, Hq, Hkv, d, page_size, num_pages, max_context_len,
                                  status_flag, stream, options, nullptr);
}

int ac_paged_decode_attn_ex(const void* q_rot, const void* k_cache, const void* v_cache,
                            int64_t stride_page, int64_t stride_token, int64_t stride_head,
                            const int32_t* block_table, int max_pages_per_seq,
                            const int32_t* context_lens, int new_tokens, float softmax_scale,
                            int num_splits, void* workspace, size_t workspace_bytes, void* out, int B,
                            int Hq, int Hkv, int d, int page_size, int num_pages, int max_context_len,
                            int32_t* status_flag, void* stream, const ac_attn_options* options) {
    const bool fused = options != nullptr && options->fused_merge != 0;
    const int window = options != nullptr ? options->window : 0;
    const int32_t* row_order = options != nullptr ? options->row_order : nullptr;
    return attn_common(q_rot, k_cache, v_cache, stride_page, stride_token, stride_head, block_table,
                       max_pages_per_seq, context_lens, new_tokens, softmax_scale, num_splits, workspace,
                       workspace_bytes, out, B, Hq, Hkv, d, page_size, num_pages, max_context_len,
                       status_flag, stream, fused, nullptr, window, row_order);
}

int ac_splitkv_merge(const void* workspace, int num_splits, const int32_t* context_lens, void* out,
                     int B, int Hq, int d, void* stream) {
    if (!workspace || !out) return AC_ERR_NULL;
    if (B <= 0 || Hq <= 0 || num_splits <= 0) return AC_ERR_SHAPE;
    if (d != 64 && d != 128) return AC_ERR_UNSUPPORTED;
    if (B > 65535) return AC_ERR_UNSUPPORTED;
    if (!aligned16(workspace) || !aligned16(out)) return AC_ERR_ALIGN;
    int dev;
    int st = current_ready_device(&dev);
    if (st != AC_OK) return st;
    const float* partial_o = static_cast<const float*>(workspace);
    const float* partial_lse = partial_o + static_cast<size_t>(B) * Hq * num_splits * d;
    cudaError_t e = launch_splitkv_merge(partial_o, partial_lse, num_splits, context_lens, out, B, Hq, d,
                                         static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AC_OK : fail_cuda(static_cast<int>(e));
}

int ac_decode_step_host(const void* q_host, const void* k_new_host, const void* v_new_host,
                        const int32_t* block_table_host, const int32_t* context_lens_host,
                        void* out_host, void* q, void* k_new, void* v_new, int32_t* block_table,
                        int32_t* context_lens, void* out, void* k_cache, void* v_cache,
                        int64_t stride_page, int64_t stride_token, int64_t stride_head,
                        int max_pages_per_seq, const float* rope_cos, const float* rope_sin,
                        int max_position, float softmax_scale, int num_splits, void* workspace,
                        size_t workspace_bytes, int B, int Hq, int Hkv, int d, int page_size,
                        int num_pages, int max_context_len, int32_t* status_flag, void* stream) {
    if (!q_host || !k_new_host || !v_new_host || !block_table_host || !context_lens_host || !out_host ||
        !q || !k_new || !v_new || !block_table || !context_lens || !out)
        return AC_ERR_NULL;
    Shape s{B, Hq, Hkv, d, page_size, num_pages};
    int st = check_shape(s);
    if (st != AC_OK) return st;
    if (max_pages_per_seq <= 0) return AC_ERR_SHAPE;
    if (num_splits > 1 &&
        (!workspace || workspace_bytes < ac_fused_workspace_bytes(B, Hq, Hkv, d, num_splits)))
        return AC_ERR_WORKSPACE;
    int dev;
    st = current_ready_device(&dev);
    if (st != AC_OK) return st;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const size_t q_bytes = static_cast<size_t>(B) * Hq * d * 2;
    const size_t kv_bytes = static_cast<size_t>(B) * Hkv * d * 2;
    const size_t bt_bytes = static_cast<size_t>(B) * max_pages_per_seq * sizeof(int32_t);
    const size_t len_bytes = static_cast<size_t>(B) * sizeof(int32_t);
    cudaError_t e = cudaErrorInvalidValue;
    {
        // Preferred: one kernel gathers the five host buffers (pinned, GPU-addressable) and clears the
        // arrival counters.  Sizes that are not multiples of 16 bytes, or host memory the GPU cannot
        // address, fall back to one copy-engine transfer per buffer.
        const size_t len_padded = (len_bytes + 15) / 16 * 16, bt_padded = (bt_bytes + 15) / 16 * 16;
        const bool tails_ok = len_padded == len_bytes && bt_padded == bt_bytes;
        if (tails_ok) {
            const void* src[5] = {q_host, k_new_host, v_new_host, block_table_host, context_lens_host};
            void* dst[5] = {q, k_new, v_new, block_table, context_lens};
            const size_t bytes[5] = {q_bytes, kv_bytes, kv_bytes, bt_bytes, len_bytes};
            void* zero_dst = nullptr;
            size_t zero_bytes = 0;
            if (num_splits > 1) {
                // counters follow the partials; clear from the 16-byte boundary at or below their start
                // (the bytes before it belong to partial_lse, which every launch rewrites before use)
                const size_t off = ac_workspace_bytes(B, Hq, d, num_splits);
                const size_t lo = off / 16 * 16;
                const size_t hi = (off + static_cast<size_t>(B) * Hkv * sizeof(int32_t) + 15) / 16 * 16;
                if (hi <= workspace_bytes) {
                    zero_dst = static_cast<char*>(workspace) + lo;
                    zero_bytes = hi - lo;
                }
            }
            if (num_splits == 1 || zero_dst != nullptr)
                e = launch_stage_inputs(src, dst, bytes, zero_dst, zero_bytes, cs);
        }
    }
    if (e != cudaSuccess) {
        cudaGetLastError();
        st = ac_fused_workspace_reset(workspace, workspace_bytes, B, Hq, Hkv, d, num_splits, stream);
        if (st != AC_OK) return st;
        if ((e = cudaMemcpyAsync(q, q_host, q_bytes, cudaMemcpyHostToDevice, cs)) != cudaSuccess ||
            (e = cudaMemcpyAsync(k_new, k_new_host, kv_bytes, cudaMemcpyHostToDevice, cs)) != cudaSuccess ||
            (e = cudaMemcpyAsync(v_new, v_new_host, kv_bytes, cudaMemcpyHostToDevice, cs)) != cudaSuccess ||
            (e = cudaMemcpyAsync(block_table, block_table_host, bt_bytes, cudaMemcpyHostToDevice, cs)) != cudaSuccess ||
            (e = cudaMemcpyAsync(context_lens, context_lens_host, len_bytes, cudaMemcpyHostToDevice, cs)) != cudaSuccess)
            return fail_cuda(static_cast<int>(e));
    }
    // The result goes to out and, when out_host is pinned memory the GPU can address (16-byte aligned),
    // straight to out_host as well: the kernel's final stores are mirrored there, which saves the
    // device-to-host copy and the two stream hand-overs around it.  Otherwise a copy follows.
    void* mirror = nullptr;
    {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, out_host) == cudaSuccess && attr.type == cudaMemoryTypeHost &&
            attr.devicePointer != nullptr && aligned16(attr.devicePointer))
            mirror = attr.devicePointer;
        else
            cudaGetLastError();
    }
    st = decode_step_fused_impl(q, nullptr, k_new, v_new, k_cache, v_cache, stride_page, stride_token,
                                stride_head, block_table, max_pages_per_seq, context_lens, rope_cos,
                                rope_sin, max_position, softmax_scale, num_splits, workspace,
                                workspace_bytes, out, B, Hq, Hkv, d, page_size, num_pages, max_context_len,
                                status_flag, stream, nullptr, mirror);
    if (st != AC_OK || mirror != nullptr) return st;
    e = cudaMemcpyAsync(out_host, out, q_bytes, cudaMemcpyDeviceToHost, cs);
    return e == cudaSuccess ? AC_OK : fail_cuda(static_cast<int>(e));
}

}  // extern "C"
