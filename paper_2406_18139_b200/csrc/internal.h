// Internal declarations shared by the host planner (api.cu) and the kernel files.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/lookm.h"

namespace lookm {

constexpr int kTile = 128;      // tokens per tile on either operand of the tensor-core kernels
constexpr int kHeadDim = 128;   // only supported head_dim
constexpr int kMinUnitEntries = 32; // least number of rows in a work unit of the merge kernel
#ifndef LOOKM_MAX_UNIT_ENTRIES
#define LOOKM_MAX_UNIT_ENTRIES 256
#endif
constexpr int kMaxUnitEntries = LOOKM_MAX_UNIT_ENTRIES;   // most rows in one
// Digits of the assignment inversion's radix sort: the slot index of a request with B kept rows is
// split into the fewest digits of at most max_bits bits, all of the same width (so B <= 2^max_bits
// is sorted in one pass).  16-bit counters allow 11-bit digits, 32-bit counters 10-bit ones.
constexpr int kInvDigitBits16 = 11;
constexpr int kInvDigitBits32 = 10;
constexpr int kInvWideCountsAbove = 65535;   // evicted tokens per head beyond which counts need 32 bits
#ifdef __CUDACC__
__host__ __device__
#endif
inline void invert_digits(int B, int max_bits, int& n_pass, int& dbits) {
    int bits = 1;
    while ((1 << bits) < B) ++bits;
    n_pass = (bits + max_bits - 1) / max_bits;
    dbits = (bits + n_pass - 1) / n_pass;
}
constexpr int kMergePartBytes = 2560; // per work unit: two fp32 partial K|V rows and one bf16 K|V row

// One request of the packed batch as the kernels see it (device copy lives in the workspace).
// Requests are stored longest first so that the heaviest work items are issued first.
struct Req {
    int tok_begin;        // first token of the request on the packed token axis
    int L;                // prompt length
    int B;                // kept rows  = min(budget, L)
    int M;                // recent window, clamped to B
    int E;                // evicted rows = L - B
    int mode;             // lookm_merge_mode; LOOKM_MERGE_NONE requests have no match items and no
                          // merge work units
    int nblk;             // ceil(L / kTile)
    int out_begin;        // sum of B over the requests before this one (caller order)
    long long kept_off;   // n_kv_heads * out_begin          (start of this request's kept lists)
    long long ev_off;     // n_kv_heads * sum of E before    (start of this request's evicted lists)
    long long sim_off;    // n_kv_heads * sum of E*B before  (start of its similarity blocks)
    long long rp_off;     // kept_off + n_kv_heads * (caller index): start of its row_ptr blocks,
                          // which hold B + 1 entries per head
    int item_begin[3];    // first work item of this request in sweep 1 / sweep 2 / match order
    int slot_begin;       // first (head, slot) row of this request in merge order (table order)
    int unit_entries;     // entries read per merge work unit: chosen per call so that every warp
                          // of the merge kernel gets about one unit
    int unit_begin;       // first merge work unit of this request (table order); n_kv_heads *
                          // ceil(L / unit_entries) units per request, heads varying fastest
};

enum TileKind { kSweep1 = 0, kSweep2 = 1, kMatch = 2 };

struct TileParams {
    const Req* reqs;
    int n_req;
    int n_items;
    int n_q_heads, n_kv_heads, group;
    long long T;                 // total packed tokens
    float scale_log2;            // softmax scale * log2(e)
    float* lse;                  // [n_q_heads, T] natural log (sweep 1 writes)
    unsigned short* lse_split;   // [T, n_q_heads, 16] bf16: -lse / scale as three bf16 terms and 13
                                 // zeros per query row (sweep 1 writes, sweep 2 loads it by TMA)
    float* scores;               // [n_kv_heads, T]
    const int* evict_idx;        // evicted-list layout  (match: rows of the stationary tiles)
    const void* k_rows;          // K [tokens, heads, 128] bf16 with the strides below (match)
    long long k_stride_tok, k_stride_head;
    const float* rnorm_all;      // [n_kv_heads, T]      (match)
    const float* rnorm_kept;     // kept-list layout     (match)
    int* assign;                 // evicted-list layout  (match)
    float* sim;                  // evicted-list layout  (match)
    int* status;                 // device status word
};

// ---- launchers (each enqueues on `stream` and returns the CUDA error of the launch) -----------
// map_x: the lse_split tensor (sweep 2 only; NULL otherwise)
cudaError_t launch_tile_kernel(int kind, const CUtensorMap& map_a, const CUtensorMap& map_b,
                               const CUtensorMap* map_x, const TileParams& p, int num_sms,
                               cudaStream_t stream);

// lse_split from a given lse (for callers that supply their own log-sum-exp)
cudaError_t launch_lse_split(const float* lse, int n_q_heads, long long T, float scale_log2,
                             unsigned short* lse_split, cudaStream_t stream);

// One CTA that waits, with the tile kernels' own bounded wait and the given limit, on an mbarrier
// nobody arrives at; on expiry it writes LOOKM_ERR_DEVICE_TIMEOUT to *status like they do.
cudaError_t launch_wait_probe(unsigned long long limit_ns, int* status, cudaStream_t stream);

cudaError_t launch_select(const float* scores, const uint8_t* mask, const Req* reqs, int n_req,
                          int n_kv_heads, long long T, int* kept_idx, int* evict_idx, int* rank,
                          const void* k_for_norms, long long stride_tok, long long stride_head,
                          float* rnorm_all, int num_sms, cudaStream_t stream);

cudaError_t launch_key_norms(const void* k, long long stride_tok, long long stride_head,
                             int n_kv_heads, long long T, float* rnorm_all, cudaStream_t stream);

cudaError_t launch_gather_kept(const void* k, long long stride_tok, long long stride_head,
                               const Req* reqs, int n_req, int n_kv_heads, long long T,
                               long long total_kept_rows, const int* kept_idx,
                               const float* rnorm_all, void* kept_keys, float* rnorm_kept,
                               int* status, cudaStream_t stream);

cudaError_t launch_argmax_rows(const float* sim_matrix, const Req* reqs, int n_req, int n_kv_heads,
                               int max_evicted, int* assign, float* sim, cudaStream_t stream);

// Copies up to kReqChunk table entries, passed by value as a kernel argument, into the workspace;
// this keeps the host free of any synchronising copy.
constexpr int kReqChunk = 40;
struct ReqChunk { Req r[kReqChunk]; };
cudaError_t launch_write_table(const ReqChunk& chunk, int count, Req* dst, cudaStream_t stream);

cudaError_t launch_invert_assignment(const int* assign, const int* kept_idx, const int* evict_idx,
                                     const float* sim, const Req* reqs, int n_req, int n_kv_heads,
                                     long long T, bool wide_counts, int digit_bits, int* row_ptr,
                                     int* ent_pos, float* ent_w, int4* unit_first, int* slot_cnt,
                                     unsigned* sort_a, unsigned* sort_b, int* status,
                                     cudaStream_t stream);

int merge_warps_per_sm();

cudaError_t launch_merge(const void* k, const void* v, long long stride_tok, long long stride_head,
                         const Req* reqs, int n_req, int n_kv_heads, long long T,
                         long long total_units, const int* row_ptr, const int* ent_pos,
                         const float* ent_w, const int4* unit_first, int* slot_cnt, float* parts,
                         int varlen_output, long long out_stride_head, void* out_k, void* out_v,
                         int* status, int num_sms, cudaStream_t stream);

// Kept K and V rows of the requests whose mode is LOOKM_MERGE_NONE copied to the output cache
// (eviction alone, Eq. 6-7); requests with another mode are left to the merge kernel.
cudaError_t launch_compact_kept(const void* k, const void* v, long long stride_tok,
                                long long stride_head, const Req* reqs, int n_req, int n_kv_heads,
                                long long total_kept_rows, const int* kept_idx, int varlen_output,
                                long long out_stride_head, void* out_k, void* out_v, int* status,
                                cudaStream_t stream);

// ---- generation step over a cache (decode_kernel.cu) --------------------------------------------
// One request of a decode call as the kernel sees it; a launch carries up to kDecodeChunk of them
// by value (no table in device memory, no copy that would synchronise the host).
struct DecodeReq {
    long long begin;      // first cache row of the request
    int len;              // cached rows before the step
    int index;            // position of the request in the caller's q / k_new / v_new / out arrays
    int n_splits;         // CTAs per (KV head, pass)
    int cta_begin;        // first CTA of the request in this launch
    int part_begin;       // first partial-result record of the request in the workspace
    int pad;
};
constexpr int kDecodeChunk = 96;
struct DecodeBatch { int n_req; int pad; DecodeReq r[kDecodeChunk]; };

#ifndef LOOKM_DEC_THREADS
#define LOOKM_DEC_THREADS 256
#endif
constexpr int kDecodeThreads = LOOKM_DEC_THREADS;             // threads per CTA of the decode kernel
constexpr int kDecodeMaxCtasPerSm = 2048 / kDecodeThreads;    // what an SM's thread limit allows
int decode_ctas_per_sm(int gt);          // resident CTAs per SM of the kernel for this gt (0: unknown)

// gt: query heads handled per pass over the rows (1, 2, 4 or 8; divides the group size)
cudaError_t launch_decode(const DecodeBatch& batch, int total_ctas, int gt, const void* q,
                          const void* k_new, const void* v_new, void* cache_k, void* cache_v,
                          long long stride_row, long long stride_head, int n_q_heads, int n_kv_heads,
                          int rows_per_split, float scale_log2, float* parts, float* out,
                          cudaStream_t stream);
// adds the splits of every request of the batch that has more than one (chained behind launch_decode)
cudaError_t launch_decode_combine(const DecodeBatch& batch, int gt, int n_q_heads, int n_kv_heads,
                                  float scale_log2, const float* parts, float* out, cudaStream_t stream);

// Function attributes (the dynamic shared-memory limit) are set once per device, not per launch:
// `mask` holds one bit per device ordinal on which `configure` has succeeded.  Two threads may both
// run `configure` the first time, which is harmless.
#ifdef __CUDACC__
template <class F>
inline cudaError_t once_per_device(unsigned long long& mask, F configure) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    const unsigned long long bit = 1ull << (dev & 63);
    if (__atomic_load_n(&mask, __ATOMIC_ACQUIRE) & bit) return cudaSuccess;
    err = configure();
    if (err == cudaSuccess) __atomic_fetch_or(&mask, bit, __ATOMIC_RELEASE);
    return err;
}
#endif

// Launch with programmatic stream serialisation: the grid may be set up while the kernel before it
// in the stream drains.  Every kernel launched this way starts with grid_dependency_wait(), which
// returns once that kernel has completed and its writes are visible (a no-op for plain launches).
#ifdef __CUDACC__
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                  cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
__device__ __forceinline__ void grid_dependency_wait() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
#endif

}  // namespace lookm
