// Host side of the C ABI: argument checks, workspace carving, the request table, TMA tensor maps
// and the launch sequence.  Nothing here synchronises with the device or allocates device memory.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <initializer_list>
#include <mutex>
#include <vector>

#include <cudaTypedefs.h>

#include "internal.h"

namespace lookm {
namespace {

thread_local int g_launches = 0;
thread_local void* const* g_stage_events = nullptr;

// Records stage event i of the caller (if per-stage timing is on); errors are ignored on purpose:
// timing must never change the result of a call.
void mark_stage(int i, cudaStream_t st) {
    if (g_stage_events && g_stage_events[i]) cudaEventRecord(static_cast<cudaEvent_t>(g_stage_events[i]), st);
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Plan {
    int n_req = 0, n_q_heads = 0, n_kv_heads = 0, group = 1;
    long long T = 0, sum_B = 0, sum_E = 0, sum_EB = 0;
    int max_L = 0, max_E = 0, max_B = 0;
    int n_none = 0;                         // requests with LOOKM_MERGE_NONE
    long long out_stride_head = 0;          // elements between heads of a single-prompt output
    int n_items[3] = {0, 0, 0};
    long long total_slots = 0;              // n_kv_heads * sum_B
    long long total_units = 0;              // merge work units
    std::vector<Req> reqs;                  // table order (longest first)
    std::vector<int> out_len;               // caller order
    // workspace offsets (bytes)
    size_t o_status, o_reqs, o_lse, o_lse_split, o_scores, o_rank, o_rnorm_all, o_kept, o_evict, o_kept_keys,
        o_rnorm_kept, o_assign, o_sim, o_row_ptr, o_members, o_member_w, o_units, o_slot_cnt, o_parts, o_sort_a, o_sort_b,
        total;
};

struct DeviceInfo { int sms = 0; int cc_major = 0; bool ok = false; };
int device_info(DeviceInfo& out);

// Returns LOOKM_OK or the status describing the first bad argument.
int build_plan(Plan& pl, const lookm_layout* lay, int n_req, const int* cu_seqlens,
               const int* seq_lens, const int* budgets, const int* windows, const int* modes) {
    if (!lay || n_req <= 0 || (!cu_seqlens && !seq_lens)) return LOOKM_ERR_INVALID_ARG;
    if (lay->head_dim != kHeadDim) return LOOKM_ERR_UNSUPPORTED;
    if (lay->n_kv_heads <= 0 || lay->n_q_heads <= 0 || lay->n_q_heads % lay->n_kv_heads)
        return LOOKM_ERR_INVALID_ARG;
    if (lay->n_kv_heads > 65535 || n_req > 65535) return LOOKM_ERR_UNSUPPORTED;
    pl.n_req = n_req;
    pl.n_q_heads = lay->n_q_heads;
    pl.n_kv_heads = lay->n_kv_heads;
    pl.group = lay->n_q_heads / lay->n_kv_heads;
    pl.reqs.resize(n_req);
    pl.out_len.resize(n_req);
    long long tok = 0, out = 0, ev = 0, eb = 0;
    for (int r = 0; r < n_req; ++r) {
        const long long begin = cu_seqlens ? cu_seqlens[r] : tok;
        const long long L = cu_seqlens ? (long long)cu_seqlens[r + 1] - cu_seqlens[r] : seq_lens[r];
        if (begin != tok || L <= 0 || L > (1 << 30)) return LOOKM_ERR_INVALID_ARG;
        const int budget = budgets ? budgets[r] : (int)L;
        const int window = windows ? windows[r] : 0;
        const int mode = modes ? modes[r] : 0;
        if (budget <= 0 || window < 0 || mode < 0 || mode > LOOKM_MERGE_NONE) return LOOKM_ERR_INVALID_ARG;
        if (mode == LOOKM_MERGE_NONE) ++pl.n_none;
        Req& q = pl.reqs[r];
        q.tok_begin = (int)begin;
        q.L = (int)L;
        q.B = (int)std::min<long long>(budget, L);
        q.M = std::min(window, q.B);
        q.E = q.L - q.B;
        q.mode = mode;
        q.nblk = (q.L + kTile - 1) / kTile;
        q.out_begin = (int)out;
        q.kept_off = (long long)pl.n_kv_heads * out;
        q.ev_off = (long long)pl.n_kv_heads * ev;
        q.sim_off = (long long)pl.n_kv_heads * eb;
        q.rp_off = q.kept_off + (long long)pl.n_kv_heads * r;
        pl.out_len[r] = q.B;
        tok += L;
        out += q.B;
        ev += q.E;
        eb += (long long)q.E * q.B;
        pl.max_L = std::max(pl.max_L, q.L);
        pl.max_E = std::max(pl.max_E, q.E);
        pl.max_B = std::max(pl.max_B, q.B);
    }
    pl.T = tok;
    pl.sum_B = out;
    pl.sum_E = ev;
    pl.sum_EB = eb;
    pl.total_slots = (long long)pl.n_kv_heads * out;
    if (pl.T + kTile >= (1ll << 31) || pl.total_slots + kTile >= (1ll << 31) ||
        (long long)pl.n_q_heads * ((pl.T + kTile - 1) / kTile + n_req) >= (1ll << 31))
        return LOOKM_ERR_UNSUPPORTED;
    // table order: longest request first
    std::stable_sort(pl.reqs.begin(), pl.reqs.end(), [](const Req& a, const Req& b) { return a.L > b.L; });
    long long it0 = 0, it1 = 0, it2 = 0, slots = 0, units = 0;
    // Merge work units (the kernel reads n_kv_heads * T rows): every warp gets the same number of
    // units, one if that keeps a unit within kMaxUnitEntries rows.  The units of a request are laid
    // out heads fastest, so a wave of warps reads one token window of all heads; with very long
    // units (a batch of many prompts) every warp would stream a far-away window of its own, and a
    // unit count just above the warp count would leave a second, nearly empty wave.
    int unit_entries = kMinUnitEntries;
    {
        DeviceInfo di;
        const int sms = (device_info(di) == LOOKM_OK && di.sms > 0) ? di.sms : 148;
        const long long per_warp = ((long long)pl.n_kv_heads * pl.T) / ((long long)sms * merge_warps_per_sm());
        if (per_warp > unit_entries) {
            const long long per_warp_units = (per_warp + kMaxUnitEntries - 1) / kMaxUnitEntries;
            const long long rows = (per_warp + per_warp_units - 1) / per_warp_units;
            unit_entries = (int)std::max<long long>(kMinUnitEntries, (rows + 7) / 8 * 8);
        }
    }
    for (Req& q : pl.reqs) {
        q.item_begin[kSweep1] = (int)it0;
        q.item_begin[kSweep2] = (int)it1;
        q.item_begin[kMatch] = (int)it2;
        q.slot_begin = (int)slots;
        q.unit_begin = (int)units;
        q.unit_entries = unit_entries;
        const bool merges = q.mode != LOOKM_MERGE_NONE;
        const long long n_units = merges ? (q.L + unit_entries - 1) / unit_entries : 0;
        units += (long long)pl.n_kv_heads * n_units;
        it0 += (long long)q.nblk * pl.n_q_heads;
        it1 += (long long)q.nblk * pl.n_kv_heads;
        // match items: blocks of 128 entries of every head's evicted list
        it2 += (q.E > 0 && merges) ? (long long)((q.E + kTile - 1) / kTile) * pl.n_kv_heads : 0;
        slots += (long long)q.B * pl.n_kv_heads;
    }
    pl.total_units = units;
    pl.n_items[kSweep1] = (int)it0;
    pl.n_items[kSweep2] = (int)it1;
    pl.n_items[kMatch] = (int)it2;

    size_t o = 0;
    auto carve = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    const size_t Hq = pl.n_q_heads, Hkv = pl.n_kv_heads, T = (size_t)pl.T;
    // Every list is sized for the worst case over budgets (at most T kept and T evicted rows per
    // head), so the carving depends only on the prompt lengths and head counts.
    pl.o_status = carve(256);
    pl.o_reqs = carve(sizeof(Req) * n_req);
    pl.o_lse = carve(4 * Hq * T);
    pl.o_lse_split = carve(32 * Hq * T);
    pl.o_scores = carve(4 * Hkv * T);
    pl.o_rank = carve(4 * Hkv * T);
    pl.o_rnorm_all = carve(4 * Hkv * T);
    pl.o_kept = carve(4 * Hkv * T);
    pl.o_evict = carve(4 * Hkv * T);
    pl.o_kept_keys = carve(2 * (size_t)kHeadDim * Hkv * T);
    pl.o_rnorm_kept = carve(4 * Hkv * T);
    pl.o_assign = carve(4 * Hkv * T);
    pl.o_sim = carve(4 * Hkv * T);
    pl.o_row_ptr = carve(4 * (Hkv * T + Hkv * (size_t)n_req));
    pl.o_members = carve(4 * Hkv * T);
    pl.o_member_w = carve(4 * Hkv * T);
    pl.o_units = carve(16 * (size_t)pl.total_units);
    pl.o_slot_cnt = carve(4 * Hkv * T);
    pl.o_parts = carve((size_t)kMergePartBytes * (size_t)pl.total_units);
    pl.o_sort_a = carve(8 * Hkv * T);
    pl.o_sort_b = carve(8 * Hkv * T);
    pl.total = o;
    return LOOKM_OK;
}

int check_layout_ptrs(const lookm_layout* lay, const void* q, const void* k, const void* v) {
    auto bad_ptr = [](const void* p) { return p && (reinterpret_cast<uintptr_t>(p) & 15u); };
    if (bad_ptr(q) || bad_ptr(k) || bad_ptr(v)) return LOOKM_ERR_INVALID_ARG;
    if (lay->q_stride_tok % 8 || lay->q_stride_head % 8 || lay->kv_stride_tok % 8 ||
        lay->kv_stride_head % 8)
        return LOOKM_ERR_INVALID_ARG;
    if (lay->q_stride_tok <= 0 || lay->q_stride_head <= 0 || lay->kv_stride_tok <= 0 ||
        lay->kv_stride_head <= 0)
        return LOOKM_ERR_INVALID_ARG;
    // the merge kernel keeps the byte stride between tokens in 32 bits
    if (lay->kv_stride_tok >= (1ll << 31)) return LOOKM_ERR_UNSUPPORTED;
    if (!(lay->softmax_scale >= 0.f) || !std::isfinite(lay->softmax_scale)) return LOOKM_ERR_INVALID_ARG;
    return LOOKM_OK;
}

int check_workspace(const Plan& pl, void* ws, size_t bytes) {
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return LOOKM_ERR_INVALID_ARG;
    if (bytes < pl.total) return LOOKM_ERR_WORKSPACE_TOO_SMALL;
    return LOOKM_OK;
}

// ---- device facts and the tensor-map encoder ---------------------------------------------------
int device_info(DeviceInfo& out) {
    static std::mutex mu;
    static DeviceInfo cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LOOKM_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!cache[dev].ok) {
        if (cudaDeviceGetAttribute(&cache[dev].sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&cache[dev].cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
            return LOOKM_ERR_CUDA;
        cache[dev].ok = true;
    }
    out = cache[dev];
    return out.cc_major == 10 ? LOOKM_OK : LOOKM_ERR_UNSUPPORTED;
}

PFN_cuTensorMapEncodeTiled_v12000 tensor_map_encoder() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
    }();
    return fn;
}

// bf16 tensor [tokens, heads, 128] with element strides; box = 128 tokens x 1 head x 64 features
// (128 bytes) with the 128-byte swizzle; out-of-range rows read as zero.
int make_map_3d(CUtensorMap* map, const void* base, long long tokens, int heads,
                long long stride_tok, long long stride_head) {
    auto enc = tensor_map_encoder();
    if (!enc) return LOOKM_ERR_CUDA;
    cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)heads, (cuuint64_t)tokens};
    cuuint64_t strides[2] = {(cuuint64_t)stride_head * 2, (cuuint64_t)stride_tok * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)kTile};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? LOOKM_OK : LOOKM_ERR_CUDA;
}

// The 16-column companion of the query tensor ([tokens, heads, 16] bf16, 32-byte rows): boxes of
// 128 tokens of one head with the 32-byte swizzle.
int make_map_split(CUtensorMap* map, const void* base, long long tokens, int heads) {
    auto enc = tensor_map_encoder();
    if (!enc) return LOOKM_ERR_CUDA;
    cuuint64_t dims[3] = {16, (cuuint64_t)heads, (cuuint64_t)tokens};
    cuuint64_t strides[2] = {32, (cuuint64_t)heads * 32};
    cuuint32_t box[3] = {16, 1, (cuuint32_t)kTile};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? LOOKM_OK : LOOKM_ERR_CUDA;
}

int make_map_2d(CUtensorMap* map, const void* base, long long rows) {
    auto enc = tensor_map_encoder();
    if (!enc) return LOOKM_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)kHeadDim * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? LOOKM_OK : LOOKM_ERR_CUDA;
}

#define LOOKM_CUDA(expr)                                  \
    do {                                                  \
        if ((expr) != cudaSuccess) return LOOKM_ERR_CUDA; \
    } while (0)
#define LOOKM_TRY(expr)                   \
    do {                                  \
        int st_ = (expr);                 \
        if (st_ != LOOKM_OK) return st_;  \
    } while (0)

template <class T>
T* at(void* ws, size_t off) { return reinterpret_cast<T*>(static_cast<char*>(ws) + off); }

// Clears the status word and writes the request table into the workspace.
int begin_call(const Plan& pl, void* ws, cudaStream_t st) {
    g_launches = 0;
    LOOKM_CUDA(cudaMemsetAsync(at<int>(ws, pl.o_status), 0, 256, st));
    for (int base = 0; base < pl.n_req; base += kReqChunk) {
        ReqChunk chunk;
        const int cnt = std::min(kReqChunk, pl.n_req - base);
        std::memset(&chunk, 0, sizeof(chunk));
        std::memcpy(chunk.r, pl.reqs.data() + base, sizeof(Req) * cnt);
        LOOKM_CUDA(launch_write_table(chunk, cnt, at<Req>(ws, pl.o_reqs) + base, st));
        ++g_launches;
    }
    return LOOKM_OK;
}

float scale_log2(const lookm_layout* lay) {
    const float s = lay->softmax_scale > 0.f ? lay->softmax_scale : 1.0f / std::sqrt((float)lay->head_dim);
    return s * 1.4426950408889634f;
}

TileParams tile_params(const Plan& pl, void* ws, const lookm_layout* lay) {
    TileParams p;
    std::memset(&p, 0, sizeof(p));
    p.reqs = at<Req>(ws, pl.o_reqs);
    p.n_req = pl.n_req;
    p.n_q_heads = pl.n_q_heads;
    p.n_kv_heads = pl.n_kv_heads;
    p.group = pl.group;
    p.T = pl.T;
    p.scale_log2 = scale_log2(lay);
    p.status = at<int>(ws, pl.o_status);
    return p;
}

int run_score(const Plan& pl, const DeviceInfo& di, const lookm_layout* lay, const void* q,
              const void* k, float* scores, float* lse, bool lse_is_input, void* ws, cudaStream_t st) {
    CUtensorMap map_q, map_k;
    LOOKM_TRY(make_map_3d(&map_q, q, pl.T, pl.n_q_heads, lay->q_stride_tok, lay->q_stride_head));
    LOOKM_TRY(make_map_3d(&map_k, k, pl.T, pl.n_kv_heads, lay->kv_stride_tok, lay->kv_stride_head));
    CUtensorMap map_x;
    unsigned short* split = at<unsigned short>(ws, pl.o_lse_split);
    LOOKM_TRY(make_map_split(&map_x, split, pl.T, pl.n_q_heads));
    TileParams p = tile_params(pl, ws, lay);
    p.lse = lse;
    p.lse_split = split;
    p.scores = scores;
    if (!lse_is_input) {
        p.n_items = pl.n_items[kSweep1];
        LOOKM_CUDA(launch_tile_kernel(kSweep1, map_q, map_k, nullptr, p, di.sms, st));
        ++g_launches;
    } else {
        LOOKM_CUDA(launch_lse_split(lse, pl.n_q_heads, pl.T, p.scale_log2, split, st));
        ++g_launches;
    }
    mark_stage(1, st);
    p.n_items = pl.n_items[kSweep2];
    LOOKM_CUDA(launch_tile_kernel(kSweep2, map_k, map_q, &map_x, p, di.sms, st));
    ++g_launches;
    mark_stage(2, st);
    return LOOKM_OK;
}

// norms_done: 1 / |k| of every key row is already in the workspace (written by the selection launch)
int run_match(const Plan& pl, const DeviceInfo& di, const lookm_layout* lay, const void* k,
              const int* kept_idx, const int* evict_idx, int* assign, float* sim, void* ws,
              bool norms_done, cudaStream_t st) {
    if (pl.n_items[kMatch] == 0) { mark_stage(4, st); mark_stage(5, st); return LOOKM_OK; }
    float* rnorm_all = at<float>(ws, pl.o_rnorm_all);
    float* rnorm_kept = at<float>(ws, pl.o_rnorm_kept);
    void* kept_keys = at<void>(ws, pl.o_kept_keys);
    const Req* reqs = at<Req>(ws, pl.o_reqs);
    if (!norms_done) {
        LOOKM_CUDA(launch_key_norms(k, lay->kv_stride_tok, lay->kv_stride_head, pl.n_kv_heads, pl.T,
                                    rnorm_all, st));
        ++g_launches;
    }
    LOOKM_CUDA(launch_gather_kept(k, lay->kv_stride_tok, lay->kv_stride_head, reqs, pl.n_req,
                                  pl.n_kv_heads, pl.T, pl.total_slots, kept_idx, rnorm_all,
                                  kept_keys, rnorm_kept, at<int>(ws, pl.o_status), st));
    ++g_launches;
    mark_stage(4, st);
    CUtensorMap map_c;                           // the evicted rows are gathered, not tiled
    LOOKM_TRY(make_map_2d(&map_c, kept_keys, pl.total_slots));
    TileParams p = tile_params(pl, ws, lay);
    p.n_items = pl.n_items[kMatch];
    p.evict_idx = evict_idx;
    p.k_rows = k;
    p.k_stride_tok = lay->kv_stride_tok;
    p.k_stride_head = lay->kv_stride_head;
    p.rnorm_all = rnorm_all;
    p.rnorm_kept = rnorm_kept;
    p.assign = assign;
    p.sim = sim;
    LOOKM_CUDA(launch_tile_kernel(kMatch, map_c, map_c, nullptr, p, di.sms, st));
    ++g_launches;
    mark_stage(5, st);
    return LOOKM_OK;
}

int run_merge(const Plan& pl, const lookm_layout* lay, const void* k, const void* v,
              const int* kept_idx, const int* evict_idx, const int* assign, const float* sim,
              int varlen_output, void* out_k, void* out_v, void* ws, cudaStream_t st) {
    const Req* reqs = at<Req>(ws, pl.o_reqs);
    int* status = at<int>(ws, pl.o_status);
    if (pl.n_none < pl.n_req) {
        // counter width and widest digit over the requests of the call
        const bool wide = pl.max_E > kInvWideCountsAbove;
        int digit_bits = 1;
        for (const Req& r : pl.reqs) {
            int n_pass, dbits;
            invert_digits(r.B, wide ? kInvDigitBits32 : kInvDigitBits16, n_pass, dbits);
            digit_bits = std::max(digit_bits, dbits);
        }
        LOOKM_CUDA(launch_invert_assignment(assign, kept_idx, evict_idx, sim, reqs, pl.n_req, pl.n_kv_heads,
                                            pl.T, wide, digit_bits, at<int>(ws, pl.o_row_ptr), at<int>(ws, pl.o_members),
                                            at<float>(ws, pl.o_member_w), at<int4>(ws, pl.o_units),
                                            at<int>(ws, pl.o_slot_cnt), at<unsigned>(ws, pl.o_sort_a),
                                            at<unsigned>(ws, pl.o_sort_b), status, st));
        ++g_launches;
    }
    mark_stage(6, st);
    if (pl.n_none < pl.n_req) {
        DeviceInfo di;
        LOOKM_TRY(device_info(di));
        LOOKM_CUDA(launch_merge(k, v, lay->kv_stride_tok, lay->kv_stride_head, reqs, pl.n_req,
                                pl.n_kv_heads, pl.T, pl.total_units, at<int>(ws, pl.o_row_ptr),
                                at<int>(ws, pl.o_members), at<float>(ws, pl.o_member_w),
                                at<int4>(ws, pl.o_units), at<int>(ws, pl.o_slot_cnt),
                                at<float>(ws, pl.o_parts), varlen_output, pl.out_stride_head, out_k,
                                out_v, status, di.sms, st));
        ++g_launches;
    }
    if (pl.n_none > 0) {
        // eviction alone: the kept rows of those requests go straight to the output
        LOOKM_CUDA(launch_compact_kept(k, v, lay->kv_stride_tok, lay->kv_stride_head, reqs, pl.n_req,
                                       pl.n_kv_heads, pl.total_slots, kept_idx, varlen_output,
                                       pl.out_stride_head, out_k, out_v, status, st));
        ++g_launches;
    }
    mark_stage(7, st);
    return LOOKM_OK;
}

// Output pointers are written with 16-byte stores, index and weight lists read as 32-bit words.
int check_out_ptrs(const void* out_k, const void* out_v) {
    if ((reinterpret_cast<uintptr_t>(out_k) & 15u) || (reinterpret_cast<uintptr_t>(out_v) & 15u))
        return LOOKM_ERR_INVALID_ARG;
    return LOOKM_OK;
}
int check_word_ptrs(std::initializer_list<const void*> ptrs) {
    for (const void* p : ptrs)
        if (reinterpret_cast<uintptr_t>(p) & 3u) return LOOKM_ERR_INVALID_ARG;
    return LOOKM_OK;
}

// Stride between the heads of a single-prompt output (0 = dense).
int set_out_stride(Plan& pl, int varlen_output, long long out_stride_head) {
    pl.out_stride_head = 0;
    if (varlen_output) return out_stride_head ? LOOKM_ERR_INVALID_ARG : LOOKM_OK;
    const long long dense = (long long)pl.out_len[0] * kHeadDim;
    if (out_stride_head == 0) { pl.out_stride_head = dense; return LOOKM_OK; }
    if (out_stride_head % 8 || out_stride_head < dense) return LOOKM_ERR_INVALID_ARG;
    pl.out_stride_head = out_stride_head;
    return LOOKM_OK;
}

int compress_common(const void* q, const void* k, const void* v, const uint8_t* mask,
                    const int* cu_seqlens, int n_req, const int* budgets, const int* windows,
                    const int* modes, const lookm_layout* lay, const lookm_options* opt,
                    int varlen_output, void* out_k, void* out_v, int* out_cu, void* ws,
                    size_t ws_bytes, void* stream) {
    const unsigned flags = opt ? opt->flags : 0u;
    const float* lse_in = opt ? opt->lse : nullptr;
    if (flags & ~LOOKM_OPT_NO_TEXT_PRIOR) return LOOKM_ERR_INVALID_ARG;
    const bool text_prior = !(flags & LOOKM_OPT_NO_TEXT_PRIOR);
    if (!q || !k || !v || (!mask && text_prior) || !out_k || !out_v || !budgets || !windows || !modes)
        return LOOKM_ERR_INVALID_ARG;
    Plan pl;
    LOOKM_TRY(build_plan(pl, lay, n_req, cu_seqlens, nullptr, budgets, windows, modes));
    LOOKM_TRY(check_layout_ptrs(lay, q, k, v));
    LOOKM_TRY(check_out_ptrs(out_k, out_v));
    LOOKM_TRY(check_word_ptrs({lse_in}));
    LOOKM_TRY(set_out_stride(pl, varlen_output, opt ? opt->out_stride_head : 0));
    LOOKM_TRY(check_workspace(pl, ws, ws_bytes));
    DeviceInfo di;
    LOOKM_TRY(device_info(di));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (out_cu) {
        out_cu[0] = 0;
        for (int r = 0; r < n_req; ++r) out_cu[r + 1] = out_cu[r] + pl.out_len[r];
    }
    LOOKM_TRY(begin_call(pl, ws, st));
    mark_stage(0, st);
    float* scores = at<float>(ws, pl.o_scores);
    int* kept = at<int>(ws, pl.o_kept);
    int* evict = at<int>(ws, pl.o_evict);
    int* rank = at<int>(ws, pl.o_rank);
    int* assign = at<int>(ws, pl.o_assign);
    float* sim = at<float>(ws, pl.o_sim);
    // a caller's log-sum-exp (read only) replaces the first sweep
    float* lse = lse_in ? const_cast<float*>(lse_in) : at<float>(ws, pl.o_lse);
    LOOKM_TRY(run_score(pl, di, lay, q, k, scores, lse, lse_in != nullptr, ws, st));
    // the selection launch also computes the key norms that the matching needs
    const bool need_match = pl.n_items[kMatch] > 0;
    LOOKM_CUDA(launch_select(scores, text_prior ? mask : nullptr, at<Req>(ws, pl.o_reqs), pl.n_req,
                             pl.n_kv_heads, pl.T, kept, evict, rank, need_match ? k : nullptr,
                             lay->kv_stride_tok, lay->kv_stride_head, at<float>(ws, pl.o_rnorm_all),
                             di.sms, st));
    ++g_launches;
    mark_stage(3, st);
    LOOKM_TRY(run_match(pl, di, lay, k, kept, evict, assign, sim, ws, true, st));
    LOOKM_TRY(run_merge(pl, lay, k, v, kept, evict, assign, sim, varlen_output, out_k, out_v, ws, st));
    return LOOKM_OK;
}

}  // namespace
}  // namespace lookm

using namespace lookm;

extern "C" {

size_t lookm_workspace_size(const lookm_layout* layout, int n_requests, const int* seq_lens_host,
                            const int* budgets_host) {
    Plan pl;
    if (!seq_lens_host) return 0;
    if (build_plan(pl, layout, n_requests, nullptr, seq_lens_host, budgets_host, nullptr, nullptr) != LOOKM_OK)
        return 0;
    return pl.total;
}

int lookm_workspace_layout(const lookm_layout* layout, int n_requests, const int* seq_lens_host,
                           lookm_workspace_offsets* offsets_host) {
    Plan pl;
    if (!seq_lens_host || !offsets_host) return LOOKM_ERR_INVALID_ARG;
    LOOKM_TRY(build_plan(pl, layout, n_requests, nullptr, seq_lens_host, nullptr, nullptr, nullptr));
    offsets_host->status = pl.o_status;
    offsets_host->lse = pl.o_lse;
    offsets_host->scores = pl.o_scores;
    offsets_host->rank = pl.o_rank;
    offsets_host->kept_idx = pl.o_kept;
    offsets_host->evict_idx = pl.o_evict;
    offsets_host->assign = pl.o_assign;
    offsets_host->sim = pl.o_sim;
    return LOOKM_OK;
}

int lookm_compress_layer_opt(const void* q, const void* k, const void* v, const uint8_t* modality_mask,
                             int seq_len, int budget, int recent_window, int merge_mode,
                             const lookm_layout* layout, const lookm_options* options, void* out_k,
                             void* out_v, int* out_len_host, void* workspace, size_t workspace_bytes,
                             void* cuda_stream) {
    if (seq_len <= 0) return LOOKM_ERR_INVALID_ARG;
    const int cu[2] = {0, seq_len};
    int out_cu[2] = {0, 0};
    const int st = compress_common(q, k, v, modality_mask, cu, 1, &budget, &recent_window, &merge_mode,
                                   layout, options, 0, out_k, out_v, out_cu, workspace, workspace_bytes,
                                   cuda_stream);
    if (st == LOOKM_OK && out_len_host) *out_len_host = out_cu[1];
    return st;
}

int lookm_compress_layer(const void* q, const void* k, const void* v, const uint8_t* modality_mask,
                         int seq_len, int budget, int recent_window, int merge_mode,
                         const lookm_layout* layout, void* out_k, void* out_v, int* out_len_host,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return lookm_compress_layer_opt(q, k, v, modality_mask, seq_len, budget, recent_window, merge_mode,
                                    layout, nullptr, out_k, out_v, out_len_host, workspace,
                                    workspace_bytes, cuda_stream);
}

int lookm_compress_varlen_opt(const void* q, const void* k, const void* v, const uint8_t* modality_mask,
                              const int* cu_seqlens_host, int n_requests, const int* budgets_host,
                              const int* windows_host, const int* merge_modes_host,
                              const lookm_layout* layout, const lookm_options* options, void* out_k,
                              void* out_v, int* out_cu_seqlens_host, void* workspace,
                              size_t workspace_bytes, void* cuda_stream) {
    if (!cu_seqlens_host) return LOOKM_ERR_INVALID_ARG;
    return compress_common(q, k, v, modality_mask, cu_seqlens_host, n_requests, budgets_host,
                           windows_host, merge_modes_host, layout, options, 1, out_k, out_v,
                           out_cu_seqlens_host, workspace, workspace_bytes, cuda_stream);
}

int lookm_compress_varlen(const void* q, const void* k, const void* v, const uint8_t* modality_mask,
                          const int* cu_seqlens_host, int n_requests, const int* budgets_host,
                          const int* windows_host, const int* merge_modes_host,
                          const lookm_layout* layout, void* out_k, void* out_v,
                          int* out_cu_seqlens_host, void* workspace, size_t workspace_bytes,
                          void* cuda_stream) {
    return lookm_compress_varlen_opt(q, k, v, modality_mask, cu_seqlens_host, n_requests, budgets_host,
                                     windows_host, merge_modes_host, layout, nullptr, out_k, out_v,
                                     out_cu_seqlens_host, workspace, workspace_bytes, cuda_stream);
}

int lookm_score(const void* q, const void* k, const int* cu_seqlens_host, int n_requests,
                const lookm_layout* layout, float* scores, float* lse, int lse_is_input,
                void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!q || !k || !cu_seqlens_host || !scores || (lse_is_input && !lse)) return LOOKM_ERR_INVALID_ARG;
    LOOKM_TRY(check_word_ptrs({scores, lse}));
    Plan pl;
    LOOKM_TRY(build_plan(pl, layout, n_requests, cu_seqlens_host, nullptr, nullptr, nullptr, nullptr));
    LOOKM_TRY(check_layout_ptrs(layout, q, k, nullptr));
    LOOKM_TRY(check_workspace(pl, workspace, workspace_bytes));
    DeviceInfo di;
    LOOKM_TRY(device_info(di));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    LOOKM_TRY(begin_call(pl, workspace, st));
    float* lse_buf = lse ? lse : at<float>(workspace, pl.o_lse);
    return run_score(pl, di, layout, q, k, scores, lse_buf, lse_is_input != 0, workspace, st);
}

int lookm_select(const float* scores, const uint8_t* modality_mask, const int* cu_seqlens_host,
                 int n_requests, const int* budgets_host, const int* windows_host, int n_kv_heads,
                 int* kept_idx, int* evict_idx, int* rank, void* workspace, size_t workspace_bytes,
                 void* cuda_stream) {
    if (!scores || !cu_seqlens_host || !budgets_host || !windows_host || !kept_idx || !evict_idx)
        return LOOKM_ERR_INVALID_ARG;
    LOOKM_TRY(check_word_ptrs({scores, kept_idx, evict_idx, rank}));
    lookm_layout lay;
    std::memset(&lay, 0, sizeof(lay));
    lay.n_q_heads = lay.n_kv_heads = n_kv_heads;
    lay.head_dim = kHeadDim;
    Plan pl;
    LOOKM_TRY(build_plan(pl, &lay, n_requests, cu_seqlens_host, nullptr, budgets_host, windows_host, nullptr));
    LOOKM_TRY(check_workspace(pl, workspace, workspace_bytes));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    LOOKM_TRY(begin_call(pl, workspace, st));
    LOOKM_CUDA(launch_select(scores, modality_mask, at<Req>(workspace, pl.o_reqs), pl.n_req,
                             pl.n_kv_heads, pl.T, kept_idx, evict_idx, rank, nullptr, 0, 0, nullptr, 0, st));
    ++g_launches;
    return LOOKM_OK;
}

int lookm_match(const void* k, const int* kept_idx, const int* evict_idx, const int* cu_seqlens_host,
                int n_requests, const int* budgets_host, const lookm_layout* layout, int* assign,
                float* sim, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!k || !kept_idx || !evict_idx || !cu_seqlens_host || !budgets_host || !assign || !sim)
        return LOOKM_ERR_INVALID_ARG;
    LOOKM_TRY(check_word_ptrs({kept_idx, evict_idx, assign, sim}));
    Plan pl;
    LOOKM_TRY(build_plan(pl, layout, n_requests, cu_seqlens_host, nullptr, budgets_host, nullptr, nullptr));
    LOOKM_TRY(check_layout_ptrs(layout, nullptr, k, nullptr));
    LOOKM_TRY(check_workspace(pl, workspace, workspace_bytes));
    DeviceInfo di;
    LOOKM_TRY(device_info(di));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    LOOKM_TRY(begin_call(pl, workspace, st));
    return run_match(pl, di, layout, k, kept_idx, evict_idx, assign, sim, workspace, false, st);
}

int lookm_match_from_sim(const float* sim_matrix, const int* cu_seqlens_host, int n_requests,
                         const int* budgets_host, int n_kv_heads, int* assign, float* sim,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!sim_matrix || !cu_seqlens_host || !budgets_host || !assign || !sim) return LOOKM_ERR_INVALID_ARG;
    LOOKM_TRY(check_word_ptrs({sim_matrix, assign, sim}));
    lookm_layout lay;
    std::memset(&lay, 0, sizeof(lay));
    lay.n_q_heads = lay.n_kv_heads = n_kv_heads;
    lay.head_dim = kHeadDim;
    Plan pl;
    LOOKM_TRY(build_plan(pl, &lay, n_requests, cu_seqlens_host, nullptr, budgets_host, nullptr, nullptr));
    LOOKM_TRY(check_workspace(pl, workspace, workspace_bytes));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    LOOKM_TRY(begin_call(pl, workspace, st));
    LOOKM_CUDA(launch_argmax_rows(sim_matrix, at<Req>(workspace, pl.o_reqs), pl.n_req, pl.n_kv_heads,
                                  pl.max_E, assign, sim, st));
    ++g_launches;
    return LOOKM_OK;
}

int lookm_merge(const void* k, const void* v, const int* kept_idx, const int* evict_idx,
                const int* assign, const float* sim, const int* cu_seqlens_host, int n_requests,
                const int* budgets_host, const int* merge_modes_host, const lookm_layout* layout,
                int varlen_output, void* out_k, void* out_v, void* workspace,
                size_t workspace_bytes, void* cuda_stream) {
    if (!k || !v || !kept_idx || !evict_idx || !cu_seqlens_host || !budgets_host || !merge_modes_host ||
        !out_k || !out_v)
        return LOOKM_ERR_INVALID_ARG;
    if (!varlen_output && n_requests != 1) return LOOKM_ERR_INVALID_ARG;
    Plan pl;
    LOOKM_TRY(build_plan(pl, layout, n_requests, cu_seqlens_host, nullptr, budgets_host, nullptr,
                         merge_modes_host));
    if ((!assign || !sim) && pl.n_none < pl.n_req) return LOOKM_ERR_INVALID_ARG;
    LOOKM_TRY(check_layout_ptrs(layout, nullptr, k, v));
    LOOKM_TRY(check_out_ptrs(out_k, out_v));
    LOOKM_TRY(check_word_ptrs({kept_idx, evict_idx, assign, sim}));
    LOOKM_TRY(set_out_stride(pl, varlen_output, 0));
    LOOKM_TRY(check_workspace(pl, workspace, workspace_bytes));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    LOOKM_TRY(begin_call(pl, workspace, st));
    return run_merge(pl, layout, k, v, kept_idx, evict_idx, assign, sim, varlen_output, out_k, out_v,
                     workspace, st);
}

int lookm_device_status(void* workspace, void* cuda_stream) {
    if (!workspace) return LOOKM_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int word = 0;
    if (cudaStreamSynchronize(st) != cudaSuccess) return LOOKM_ERR_CUDA;
    if (cudaMemcpy(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return LOOKM_ERR_CUDA;
    if (word != 0 && cudaMemset(workspace, 0, sizeof(int)) != cudaSuccess) return LOOKM_ERR_CUDA;
    return word;
}

int lookm_selftest_wait_expiry(int limit_us, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (limit_us < 1 || limit_us > 100000) return LOOKM_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return LOOKM_ERR_INVALID_ARG;
    if (workspace_bytes < 256) return LOOKM_ERR_WORKSPACE_TOO_SMALL;
    DeviceInfo di;
    LOOKM_TRY(device_info(di));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    g_launches = 0;
    LOOKM_CUDA(cudaMemsetAsync(workspace, 0, 256, st));
    LOOKM_CUDA(launch_wait_probe(1000ull * (unsigned long long)limit_us, static_cast<int*>(workspace), st));
    ++g_launches;
    return LOOKM_OK;
}

int lookm_last_launch_count(void) { return g_launches; }

int lookm_set_stage_events(void* const* events_host, int n_events) {
    if (!events_host || n_events == 0) { g_stage_events = nullptr; return LOOKM_OK; }
    if (n_events != LOOKM_N_STAGE_EVENTS) return LOOKM_ERR_INVALID_ARG;
    g_stage_events = events_host;
    return LOOKM_OK;
}

const char* lookm_strerror(int status) {
    switch (status) {
        case LOOKM_OK: return "ok";
        case LOOKM_ERR_INVALID_ARG: return "invalid argument";
        case LOOKM_ERR_UNSUPPORTED: return "unsupported configuration or device";
        case LOOKM_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case LOOKM_ERR_CUDA: return "a CUDA call failed";
        case LOOKM_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case LOOKM_ERR_DEVICE_BAD_INDEX: return "an index list held an out-of-range entry";
        default: return "unknown status";
    }
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// lookm_merge_noalloc: the merge step with its scratch in a static device array.
// ------------------------------------------------------------------------------------------------
namespace {

// Scratch of the no-allocation merge: status word, request table, entry lists, per-slot counters,
// per-unit records and the two sort buffers.  Lives in the library's device image, so every GPU that loads the library holds
// these bytes until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[LOOKM_NOALLOC_SCRATCH_BYTES];

// Device address of the array on the current device.  The array's name is only a host-side
// handle here; kernels must be given the address cudaGetSymbolAddress returns.  Looked up once
// per device (with that device current) and cached.
int noalloc_scratch_ptr(void** out) {
    static std::mutex mu;
    static void* cache[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LOOKM_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!cache[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return LOOKM_ERR_CUDA;
        cache[dev] = p;
    }
    *out = cache[dev];
    return LOOKM_OK;
}

}  // namespace

extern "C" int lookm_merge_noalloc(const void* k, const void* v, const int* kept_idx,
                                   const int* evict_idx, const int* assign, const float* sim,
                                   const int* cu_seqlens_host, int n_requests,
                                   const int* budgets_host, const int* merge_modes_host,
                                   const lookm_layout* layout, int varlen_output, void* out_k,
                                   void* out_v, void* cuda_stream) {
    if (!k || !v || !kept_idx || !evict_idx || !assign || !sim || !cu_seqlens_host || !budgets_host ||
        !merge_modes_host || !out_k || !out_v)
        return LOOKM_ERR_INVALID_ARG;
    if (!varlen_output && n_requests != 1) return LOOKM_ERR_INVALID_ARG;
    Plan pl;
    LOOKM_TRY(build_plan(pl, layout, n_requests, cu_seqlens_host, nullptr, budgets_host, nullptr,
                         merge_modes_host));
    LOOKM_TRY(check_layout_ptrs(layout, nullptr, k, v));
    LOOKM_TRY(check_out_ptrs(out_k, out_v));
    LOOKM_TRY(check_word_ptrs({kept_idx, evict_idx, assign, sim}));
    LOOKM_TRY(set_out_stride(pl, varlen_output, 0));
    // compact carving of just what the merge needs: 28 bytes per (KV head, token), 4 per kept row,
    // the per-unit records and the table
    const size_t units = (size_t)pl.n_kv_heads * (size_t)pl.T;
    size_t o = 0;
    auto carve = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    pl.o_status = carve(256);
    pl.o_reqs = carve(sizeof(Req) * (size_t)n_requests);
    pl.o_row_ptr = carve(4 * (units + (size_t)pl.n_kv_heads * (size_t)n_requests));
    pl.o_members = carve(4 * units);
    pl.o_member_w = carve(4 * units);
    pl.o_units = carve(16 * (size_t)pl.total_units);
    pl.o_slot_cnt = carve(4 * (size_t)pl.total_slots);
    pl.o_parts = carve((size_t)kMergePartBytes * (size_t)pl.total_units);
    pl.o_sort_a = carve(8 * units);
    pl.o_sort_b = carve(8 * units);
    pl.total = o;
    if (pl.total > (size_t)LOOKM_NOALLOC_SCRATCH_BYTES) return LOOKM_ERR_WORKSPACE_TOO_SMALL;
    void* scratch = nullptr;
    LOOKM_TRY(noalloc_scratch_ptr(&scratch));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // begin_call clears the status word and rewrites the table; every list the kernels read is
    // rewritten by the inversion kernel first, so nothing else of the last call's contents matters.
    LOOKM_TRY(begin_call(pl, scratch, st));
    return run_merge(pl, layout, k, v, kept_idx, evict_idx, assign, sim, varlen_output, out_k, out_v,
                     scratch, st);
}

extern "C" int lookm_noalloc_status(void* cuda_stream) {
    void* scratch = nullptr;
    LOOKM_TRY(noalloc_scratch_ptr(&scratch));
    return lookm_device_status(scratch, cuda_stream);
}

// ------------------------------------------------------------------------------------------------
// Generation step over a cache (Section 3.1, Eq. 2-3): host planner of decode_kernel.cu.
// ------------------------------------------------------------------------------------------------
namespace {

struct DecodePlan {
    int n_req = 0, gt = 1, n_pass = 1, rows_per_split = 64;
    std::vector<DecodeReq> reqs;            // caller order
    size_t o_parts = 0, total = 0;
};

int decode_sms() {
    DeviceInfo di;
    return (device_info(di) == LOOKM_OK && di.sms > 0) ? di.sms : 148;
}

// lens may be NULL (sizing only).  The workspace is sized for the largest number of splits any
// lengths can produce, so a cache may grow from step to step under one workspace.
int build_decode_plan(DecodePlan& dp, const lookm_cache_layout* lay, int n_req, const long long* begins,
                      const int* lens) {
    if (!lay || n_req <= 0) return LOOKM_ERR_INVALID_ARG;
    if (lay->head_dim != kHeadDim) return LOOKM_ERR_UNSUPPORTED;
    if (lay->n_kv_heads <= 0 || lay->n_q_heads <= 0 || lay->n_q_heads % lay->n_kv_heads)
        return LOOKM_ERR_INVALID_ARG;
    if (lay->n_q_heads > 65535 || n_req > (1 << 20)) return LOOKM_ERR_UNSUPPORTED;
    if (lay->cache_stride_row <= 0 || lay->cache_stride_head <= 0 || lay->cache_stride_row % 8 ||
        lay->cache_stride_head % 8)
        return LOOKM_ERR_INVALID_ARG;
    if (!(lay->softmax_scale >= 0.f) || !std::isfinite(lay->softmax_scale)) return LOOKM_ERR_INVALID_ARG;
    const int group = lay->n_q_heads / lay->n_kv_heads;
    dp.n_req = n_req;
    dp.gt = group % 8 == 0 ? 8 : group % 4 == 0 ? 4 : group % 2 == 0 ? 2 : 1;
    dp.n_pass = group / dp.gt;
    const long long units = (long long)lay->n_kv_heads * dp.n_pass;      // (KV head, pass) per request
    const int sms = decode_sms();
    // The grid is one wave: as many CTAs as the GPU holds at a time (a second, partly filled wave
    // would cost as much as the first).  Rows per split: the smallest count with which the splits
    // of all requests fit into that wave.
    long long s = 16;
    if (lens) {
        const int per_sm = decode_ctas_per_sm(dp.gt);
        const long long wave = (long long)sms * (per_sm > 0 ? per_sm : 2);
        long long total_rows = 0;
        for (int r = 0; r < n_req; ++r) {
            if (lens[r] < 0 || lens[r] >= (1 << 30) || (begins && begins[r] < 0)) return LOOKM_ERR_INVALID_ARG;
            total_rows += ((long long)lens[r] + 1) * units;
        }
        auto ctas_with = [&](long long rows) {
            long long c = 0;
            for (int r = 0; r < n_req; ++r) c += (((long long)lens[r] + rows) / rows) * units;
            return c;
        };
        s = std::max<long long>(16, (total_rows + wave - 1) / wave);
        if (ctas_with(s) > wave) {
            // smallest count in (s, longest cache + 1] that fits (the CTA count never grows with
            // it); with the upper end every request is a single split, the least there can be
            long long lo = s, hi = s;
            for (int r = 0; r < n_req; ++r) hi = std::max<long long>(hi, (long long)lens[r] + 1);
            while (lo < hi) {
                const long long mid = lo + (hi - lo) / 2;
                if (ctas_with(mid) > wave) lo = mid + 1; else hi = mid;
            }
            s = lo;
        }
    }
    if (s >= (1ll << 31)) return LOOKM_ERR_UNSUPPORTED;
    dp.rows_per_split = (int)s;
    // at most one wave of the fullest kernel, or one (short) split per (request, KV head, pass)
    // when the batch alone has more units than a wave holds
    const long long max_splits = (long long)kDecodeMaxCtasPerSm * sms + (long long)n_req * units;
    if (max_splits * dp.gt >= (1ll << 31)) return LOOKM_ERR_UNSUPPORTED;
    if (lens) {
        dp.reqs.resize(n_req);
        long long parts = 0;
        for (int r = 0; r < n_req; ++r) {
            DecodeReq& q = dp.reqs[r];
            q.begin = begins ? begins[r] : 0;
            q.len = lens[r];
            q.index = r;
            q.n_splits = (int)(((long long)lens[r] + 1 + s - 1) / s);
            q.cta_begin = 0;
            q.part_begin = (int)parts;
            q.pad = 0;
            parts += (long long)q.n_splits * units * dp.gt;
        }
    }
    size_t o = 0;
    auto carve = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    dp.o_parts = carve(4 * (size_t)(kHeadDim + 2) * (size_t)max_splits * (size_t)dp.gt);
    dp.total = o;
    return LOOKM_OK;
}

int decode_common(const void* q, const void* k_new, const void* v_new, void* cache_k, void* cache_v,
                  const long long* begins, const int* lens, int n_req, const lookm_cache_layout* lay,
                  float* out, void* ws, size_t ws_bytes, void* stream) {
    if (!q || !k_new || !v_new || !cache_k || !cache_v || !lens || !out) return LOOKM_ERR_INVALID_ARG;
    for (const void* p : {q, k_new, v_new, (const void*)cache_k, (const void*)cache_v})
        if (reinterpret_cast<uintptr_t>(p) & 15u) return LOOKM_ERR_INVALID_ARG;
    LOOKM_TRY(check_word_ptrs({out}));
    DecodePlan dp;
    LOOKM_TRY(build_decode_plan(dp, lay, n_req, begins, lens));
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return LOOKM_ERR_INVALID_ARG;
    if (ws_bytes < dp.total) return LOOKM_ERR_WORKSPACE_TOO_SMALL;
    DeviceInfo di;
    LOOKM_TRY(device_info(di));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    g_launches = 0;
    const float scale = lay->softmax_scale > 0.f ? lay->softmax_scale : 1.0f / std::sqrt((float)lay->head_dim);
    const long long units = (long long)lay->n_kv_heads * dp.n_pass;
    for (int base = 0; base < n_req; base += kDecodeChunk) {
        DecodeBatch batch;
        std::memset(&batch, 0, sizeof(batch));
        batch.n_req = std::min(kDecodeChunk, n_req - base);
        long long ctas = 0;
        bool split = false;
        for (int i = 0; i < batch.n_req; ++i) {
            batch.r[i] = dp.reqs[base + i];
            batch.r[i].cta_begin = (int)ctas;
            ctas += (long long)batch.r[i].n_splits * units;
            split = split || batch.r[i].n_splits > 1;
        }
        if (ctas >= (1ll << 31)) return LOOKM_ERR_UNSUPPORTED;
        LOOKM_CUDA(launch_decode(batch, (int)ctas, dp.gt, q, k_new, v_new, cache_k, cache_v,
                                 lay->cache_stride_row, lay->cache_stride_head, lay->n_q_heads,
                                 lay->n_kv_heads, dp.rows_per_split, scale * 1.4426950408889634f,
                                 at<float>(ws, dp.o_parts), out, st));
        ++g_launches;
        if (split) {
            LOOKM_CUDA(launch_decode_combine(batch, dp.gt, lay->n_q_heads, lay->n_kv_heads,
                                             scale * 1.4426950408889634f, at<float>(ws, dp.o_parts), out, st));
            ++g_launches;
        }
    }
    return LOOKM_OK;
}

}  // namespace

extern "C" size_t lookm_decode_workspace_size(const lookm_cache_layout* layout, int n_requests,
                                              const int* cache_lens_host) {
    DecodePlan dp;
    if (build_decode_plan(dp, layout, n_requests, nullptr, cache_lens_host) != LOOKM_OK) return 0;
    return dp.total;
}

extern "C" int lookm_decode_step(const void* q, const void* k_new, const void* v_new, void* cache_k,
                                 void* cache_v, int cache_len, const lookm_cache_layout* layout,
                                 float* out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    const long long begin = 0;
    return decode_common(q, k_new, v_new, cache_k, cache_v, &begin, &cache_len, 1, layout, out, workspace,
                         workspace_bytes, cuda_stream);
}

extern "C" int lookm_decode_step_varlen(const void* q, const void* k_new, const void* v_new, void* cache_k,
                                        void* cache_v, const long long* cache_begin_host,
                                        const int* cache_lens_host, int n_requests,
                                        const lookm_cache_layout* layout, float* out, void* workspace,
                                        size_t workspace_bytes, void* cuda_stream) {
    if (!cache_begin_host) return LOOKM_ERR_INVALID_ARG;
    return decode_common(q, k_new, v_new, cache_k, cache_v, cache_begin_host, cache_lens_host, n_requests,
                         layout, out, workspace, workspace_bytes, cuda_stream);
}
