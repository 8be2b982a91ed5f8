// Tensor-core kernels of the path: the two sweeps of the cumulative attention score (Eq. 4) and
// the cosine matching with fused row argmax (Eq. 9).
//
// All three are the same persistent, warp-specialised pipeline over 128 x 128 x 128 bf16 tiles:
//   - a work item owns one STATIONARY 128-row tile (the A operand, rows on the 128 TMEM lanes)
//     and streams a sequence of 128-row tiles (the B operand) against it;
//   - warp 0 (one thread) issues the TMA loads, warps 1 and 18 (one thread each, tiles taken
//     alternately) issue tcgen05.mma into one of four 128-column TMEM accumulators, and four
//     groups of four warps read the accumulators with tcgen05.ld and run the epilogue; group w
//     owns accumulator w and takes the tiles whose running index is w mod 4, so each SM
//     sub-partition always has four epilogue warps to switch between;
//   - each epilogue thread owns one row of the stationary tile, so every reduction over the
//     streamed axis (row maximum and sum, column-sum of probabilities for one key, running
//     arg-max) stays in that thread's registers; the four groups are combined through shared
//     memory once per item.  No L x L matrix is ever stored.
//
//   sweep 1: A = 128 queries of one query head, B = key tiles 0..diagonal.  Online softmax
//            statistics per query row  ->  lse[i] = log sum_{j<=i} exp(s_ij).
//   sweep 2: A = 128 keys of one KV head, B = query tiles diagonal..last of every query head in
//            the group.  Thread of key j accumulates sum_i exp(s_ij - lse_i)  ->  A_s[j].  The
//            subtraction of lse_i is done by the tensor core: sweep 1 leaves -lse_i / scale as
//            three bf16 terms in a 16-column companion of the query tensor, and a ninth MMA per
//            tile multiplies it with a constant tile of ones, so the accumulator already holds
//            s_ij - lse_i / scale and the epilogue needs no per-column data at all.
//   match  : A = 128 EVICTED key rows in the order of the evicted list, gathered by a warp of its
//            own with 16-byte cp.async copies into the 128-byte-swizzled layout the tensor core
//            expects; B = tiles of the compacted kept keys.  Thread keeps the largest
//            s_ij / |k_j| and its slot.
//
// Work items are laid out heaviest first and dealt to the CTAs in serpentine order; every role
// walks the same item sequence on its own, so no scheduling state is shared.
#include <cuda_bf16.h>
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace lookm {
namespace {

#ifndef LOOKM_TILE_STAGES
#define LOOKM_TILE_STAGES 4
#endif
#ifndef LOOKM_TILE_ABUF
#define LOOKM_TILE_ABUF 2
#endif
constexpr int kStages = LOOKM_TILE_STAGES;       // ring of streamed tiles
constexpr int kABuf = LOOKM_TILE_ABUF;           // buffers of the stationary tile (2: the next item's is
                                                 // loaded while this item's is in use)
#ifndef LOOKM_TILE_GROUPS
#define LOOKM_TILE_GROUPS 4
#endif
constexpr int kAccum = 4;                        // TMEM accumulators (128 fp32 columns each)
#ifndef LOOKM_TILE_HALVES
#define LOOKM_TILE_HALVES 1
#endif
constexpr int kGroups = LOOKM_TILE_GROUPS;       // epilogue groups; tile g goes to group g mod kGroups
constexpr int kHalves = LOOKM_TILE_HALVES;       // a group is kHalves PARTS of four warps; part p of a group
                                                 // reads columns [p, p + 1) * kCols of the group's accumulators
constexpr int kParts = kGroups * kHalves;        // four-warp units of the epilogue (each keeps partial results)
constexpr int kCols = kTile / kHalves;           // accumulator columns per part
// "Accumulator filled" barriers form a ring twice as long as the accumulators: tile g uses barrier
// g mod kFullRing in phase g / kFullRing.  A group may reach tile g while tile g - kAccum (same
// accumulator, other group, other issuing thread) is still being multiplied; with one barrier per
// accumulator its parity wait would then pass at once.  With the longer ring the tile one phase
// back is g - 2 kAccum, whose MMAs had to complete before the producer could load tile g - kAccum,
// which it did before it loaded any tile this group has already finished.
constexpr int kFullRing = 2 * kAccum;
constexpr int kIssuers = 2;                      // MMA-issuing threads (tiles alternate between them)
constexpr int kEpiWarp0 = 2;                     // first epilogue warp
constexpr int kGatherWarp = kEpiWarp0 + kParts * 4 + 1;    // match: gathers the evicted rows of the A tiles
// producer warp, MMA warp, kParts x 4 epilogue warps, second MMA warp (+ the gather warp of the match)
__host__ __device__ constexpr int threads_of(int kind) { return 64 + kParts * 128 + 32 + (kind == kMatch ? 32 : 0); }
constexpr int kHalfBytes = kTile * 64 * 2;       // one TMA box: 128 rows x 64 bf16 (128 B rows)
constexpr int kTileBytes = 2 * kHalfBytes;       // 128 x 128 bf16
constexpr int kSplitBytes = kTile * 16 * 2;      // 128 rows x 16 bf16 (32-byte rows, 32-byte swizzle)
constexpr int kReqCache = 16;                    // request-table entries cached in shared memory
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kReferenceSlack = 1.152921504606847e18f;   // 2^60: largest chunk sum kept against a stale reference
constexpr float kLn2 = 0.6931471805599453f;

template <int KIND>
struct __align__(1024) Shared {
    static constexpr int kXStages = (KIND == kSweep2) ? kStages : 1;   // only sweep 2 streams companions
    static constexpr int kPlanes = (KIND == kSweep2) ? 1 : 2;          // values per row and part to combine
    uint8_t a[kABuf][kTileBytes];                // stationary tiles
    uint8_t b[kStages][kTileBytes];              // streamed tiles
    uint8_t bx[kXStages][kSplitBytes];           // sweep 2: the streamed tiles' 16-column companions
    union {
        float side[kParts][2][kCols];            // match: per epilogue part, double-buffered column data
        uint8_t ax[kSplitBytes];                 // sweep 2: constant ones tile that multiplies bx
    };
    float comb[2][kParts][kPlanes][kTile];       // partial results of the parts, double-buffered
    Req reqs[kReqCache];                         // copy of the request table (when it fits)
    unsigned long long a_full[kABuf], a_empty[kABuf];
    unsigned long long b_full[kStages], b_empty[kStages];
    unsigned long long t_full[2 * kAccum], t_empty[kAccum];   // t_full: see kFullRing
    unsigned long long comb_full[2], comb_free[2];   // partial results of an item written / read
    unsigned long long mma_done;                 // every MMA of this CTA has completed
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Shared<kSweep1>) + 1024 <= 232448 && sizeof(Shared<kSweep2>) + 1024 <= 232448 &&
              sizeof(Shared<kMatch>) + 1024 <= 232448, "shared memory of the tile kernels exceeds 227 KB");

// The softmax epilogues are bound by the special-function unit (16 ex2 per clock and SM), so one
// column in kPolyEvery is exponentiated on the FMA pipe instead.
constexpr int kPolyEvery = 6;
__device__ __forceinline__ float exp2_mixed(int column, float x) {
    return (column % kPolyEvery == kPolyEvery - 1) ? ptx::ex2_fma(x) : ptx::ex2(x);
}

// -lse / scale of one query row as three bf16 terms (their sum carries 24 bits) and 13 zeros:
// the row of the 16-column companion tensor that sweep 2 multiplies with ones.
__device__ __forceinline__ void store_lse_split(unsigned short* row16, float lse, float scale_log2) {
    const float u = -lse * (kLog2e / scale_log2);
    const __nv_bfloat16 hi = __float2bfloat16_rn(u);
    const float r1 = u - __bfloat162float(hi);
    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
    uint4 w0;
    w0.x = (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(mid) << 16);
    w0.y = (uint32_t)__bfloat16_as_ushort(lo);
    w0.z = 0u;
    w0.w = 0u;
    uint4* dst = reinterpret_cast<uint4*>(row16);
    dst[0] = w0;
    dst[1] = make_uint4(0u, 0u, 0u, 0u);
}

__global__ void lse_split_kernel(const float* __restrict__ lse, int n_q_heads, long long T,
                                 float scale_log2, unsigned short* __restrict__ lse_split) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // over [head][token]
    if (i >= T * n_q_heads) return;
    const long long h = i / T, tok = i % T;
    store_lse_split(lse_split + (tok * n_q_heads + h) * 16, lse[i], scale_log2);
}

struct Item {
    int tok_begin, L, B, E, blk, head, nt;
    long long kept_row0;      // match: first row of this (request, head) in the kept-key matrix
    long long ev0;            // match: start of its evicted list
};

template <int KIND>
__device__ __forceinline__ Item decode_item(const TileParams& p, const Req* tbl, int item) {
    int lo = 0, hi = p.n_req - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (tbl[mid].item_begin[KIND] <= item) lo = mid; else hi = mid - 1;
    }
    const Req& rq = tbl[lo];
    const int u = item - rq.item_begin[KIND];
    Item it;
    it.tok_begin = rq.tok_begin;
    it.L = rq.L;
    it.B = rq.B;
    it.E = rq.E;
    it.kept_row0 = 0;
    it.ev0 = 0;
    if (KIND == kSweep1) {                       // heaviest first: last query block first
        it.blk = rq.nblk - 1 - u / p.n_q_heads;
        it.head = u % p.n_q_heads;
        it.nt = it.blk + 1;
    } else if (KIND == kSweep2) {                // heaviest first: first key block first
        it.blk = u / p.n_kv_heads;
        it.head = u % p.n_kv_heads;
        it.nt = (rq.nblk - it.blk) * p.group;
    } else {                                     // blk: block of 128 entries of the evicted list
        it.blk = u / p.n_kv_heads;
        it.head = u % p.n_kv_heads;
        it.nt = (rq.B + kTile - 1) / kTile;
        it.kept_row0 = rq.kept_off + (long long)it.head * rq.B;
        it.ev0 = rq.ev_off + (long long)it.head * rq.E;
    }
    return it;
}

// Serpentine deal of the item list: round k hands items k*G .. k*G+G-1 to the CTAs in forward
// order when k is even and in reverse order when k is odd.
__device__ __forceinline__ int item_of_round(int round, int cta, int n_cta) {
    return round * n_cta + ((round & 1) ? (n_cta - 1 - cta) : cta);
}

template <int KIND>
__global__ void __launch_bounds__(threads_of(KIND), 1)
tile_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const __grid_constant__ CUtensorMap map_x, const TileParams p) {
    extern __shared__ uint8_t smem_raw[];
    Shared<KIND>& sh = *reinterpret_cast<Shared<KIND>*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    volatile int* abort_flag = &sh.abort_flag;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kABuf; ++i) {
            ptx::mbar_init(ptx::smem_u32(&sh.a_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.a_empty[i]), kIssuers);
        }
        for (int i = 0; i < kStages; ++i) {
            ptx::mbar_init(ptx::smem_u32(&sh.b_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.b_empty[i]), 1);
        }
        for (int i = 0; i < kFullRing; ++i) ptx::mbar_init(ptx::smem_u32(&sh.t_full[i]), 1);
        for (int i = 0; i < kAccum; ++i)
            ptx::mbar_init(ptx::smem_u32(&sh.t_empty[i]), 4 * kHalves);   // one arrival per epilogue warp of a group
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(ptx::smem_u32(&sh.comb_full[i]), (kParts - 1) * 4);    // warps of the other parts
            ptx::mbar_init(ptx::smem_u32(&sh.comb_free[i]), 4);                   // warps of the combining part
        }
        ptx::mbar_init(ptx::smem_u32(&sh.mma_done), kIssuers);
        sh.abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (KIND == kSweep2 && threadIdx.x < kTile) {
        // ones tile: row r = (1, 1, 1, 0, ... 0) in bf16; with the 32-byte swizzle the two 16-byte
        // halves of a row trade places in rows 4-7 of every group of eight
        const int r = threadIdx.x;
        const int first = (r >> 2) & 1;
        uint4* row = reinterpret_cast<uint4*>(sh.ax + r * 32);
        row[first] = make_uint4(0x3F803F80u, 0x00003F80u, 0u, 0u);
        row[first ^ 1] = make_uint4(0u, 0u, 0u, 0u);
        ptx::fence_proxy_async_shared();         // the tensor core reads it through the async proxy
    }
    // everything above touches only this CTA's shared memory; from here on global memory written
    // by the kernel before this one is read
    grid_dependency_wait();
    const Req* tbl = p.reqs;
    if (p.n_req <= kReqCache) {                  // the table is read once per item by every role
        for (int i = threadIdx.x; i < p.n_req * (int)(sizeof(Req) / 4); i += threads_of(KIND))
            reinterpret_cast<int*>(sh.reqs)[i] = reinterpret_cast<const int*>(p.reqs)[i];
        tbl = sh.reqs;
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&sh.tmem_base), 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = sh.tmem_base;
    const int n_cta = gridDim.x;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer ----------
        if (lane == 0) {
            ptx::prefetch_tensormap(&map_a);
            ptx::prefetch_tensormap(&map_b);
            if (KIND == kSweep2) ptx::prefetch_tensormap(&map_x);
            uint32_t gb = 0;                         // streamed tiles armed so far
            int n = 0;                               // stationary tiles armed so far
            bool stop = false;                       // a wait gave up: arm nothing more
            for (int round = 0; !stop; ++round, ++n) {
                const int item = item_of_round(round, blockIdx.x, n_cta);
                if (item >= p.n_items) { if (round * n_cta >= p.n_items) break; --n; continue; }
                const Item it = decode_item<KIND>(p, tbl, item);
                const int ab = n % kABuf;
                if (KIND != kMatch) {                    // the match's stationary tiles come from the gather warp
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.a_empty[ab]), ((n / kABuf) & 1) ^ 1, abort_flag)) break;
                    const uint32_t abar = ptx::smem_u32(&sh.a_full[ab]);
                    ptx::mbar_arrive_expect_tx(abar, kTileBytes);
                    const uint32_t adst = ptx::smem_u32(&sh.a[ab][0]);
                    const int a_head = it.head;
                    const int a_row = it.tok_begin + it.blk * kTile;
                    ptx::tma_load_3d(adst, &map_a, 0, a_head, a_row, abar);
                    ptx::tma_load_3d(adst + kHalfBytes, &map_a, 64, a_head, a_row, abar);
                }
                for (int t = 0; t < it.nt; ++t, ++gb) {
                    const int s = gb % kStages;
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.b_empty[s]), ((gb / kStages) & 1) ^ 1, abort_flag)) {
                        stop = true;
                        break;
                    }
                    const uint32_t bbar = ptx::smem_u32(&sh.b_full[s]);
                    ptx::mbar_arrive_expect_tx(bbar, KIND == kSweep2 ? kTileBytes + kSplitBytes : kTileBytes);
                    const uint32_t bdst = ptx::smem_u32(&sh.b[s][0]);
                    if (KIND == kSweep1) {
                        const int row = it.tok_begin + t * kTile;
                        const int h = it.head / p.group;
                        ptx::tma_load_3d(bdst, &map_b, 0, h, row, bbar);
                        ptx::tma_load_3d(bdst + kHalfBytes, &map_b, 64, h, row, bbar);
                    } else if (KIND == kSweep2) {
                        const int row = it.tok_begin + (it.blk + t / p.group) * kTile;
                        const int h = it.head * p.group + t % p.group;
                        ptx::tma_load_3d(bdst, &map_b, 0, h, row, bbar);
                        ptx::tma_load_3d(bdst + kHalfBytes, &map_b, 64, h, row, bbar);
                        ptx::tma_load_3d(ptx::smem_u32(&sh.bx[s % Shared<KIND>::kXStages][0]), &map_x, 0, h, row, bbar);
                    } else {
                        const int row = (int)(it.kept_row0 + (long long)t * kTile);
                        ptx::tma_load_2d(bdst, &map_b, 0, row, bbar);
                        ptx::tma_load_2d(bdst + kHalfBytes, &map_b, 64, row, bbar);
                    }
                }
            }
            // Every load issued above is consumed by an MMA before the kernel ends, except after an
            // abort.  Then nothing more was armed once a wait had given up (n and gb count exactly
            // the tiles armed), and the copies of the last ring of streamed tiles and of the last two
            // stationary tiles may still be on their way: wait for them (bounded, the flag is
            // ignored; a TMA load completes whether or not anybody consumes it), so that no copy
            // writes shared memory after the CTA has left.
            if (*abort_flag) {
                int ignore = 0;
                for (uint32_t g = (gb > (uint32_t)kStages ? gb - kStages : 0); g < gb; ++g)
                    ptx::mbar_wait(ptx::smem_u32(&sh.b_full[g % kStages]), (g / kStages) & 1, &ignore,
                                   200000000ull);
                if (KIND != kMatch)
                    for (int m = (n > kABuf ? n - kABuf : 0); m < n; ++m)
                        ptx::mbar_wait(ptx::smem_u32(&sh.a_full[m % kABuf]), (m / kABuf) & 1, &ignore, 200000000ull);
            }
        }
    } else if (KIND == kMatch && warp == kGatherWarp) {
        // ------------------------------------------------------------ gather warp (match) ---
        // Stationary tile of an item: rows e0 .. e0 + 127 of the head's evicted list, i.e. the key
        // rows at positions evict_idx[e].  Lane l copies 16-byte chunk (l mod 16) of two rows per
        // step (half a warp per 256-byte row), 64 steps per tile, into the layout a TMA box pair
        // with the 128-byte swizzle would have produced: 64 features (128 bytes) per row and box,
        // chunk c of row r at r * 128 + ((c xor (r mod 8)) * 16).  Rows past the end of the list are
        // zero-filled.  The copies are waited for and published to the tensor core's proxy before
        // the tile is announced, one item ahead of the MMAs.
        const int l16 = lane & 15;
        const int box = l16 >> 3, c8 = l16 & 7;
        int n = 0;
        for (int round = 0;; ++round, ++n) {
            const int item = item_of_round(round, blockIdx.x, n_cta);
            if (item >= p.n_items) { if (round * n_cta >= p.n_items) break; --n; continue; }
            const Item it = decode_item<KIND>(p, tbl, item);
            const int ab = n % kABuf;
            int free_now = 1;                            // one lane waits, the warp follows its verdict
            if (lane == 0)
                free_now = ptx::mbar_wait(ptx::smem_u32(&sh.a_empty[ab]), ((n / kABuf) & 1) ^ 1, abort_flag) ? 1 : 0;
            if (!__shfl_sync(0xffffffffu, free_now, 0)) break;
            const uint32_t adst = ptx::smem_u32(&sh.a[ab][0]) + box * kHalfBytes;
            const int* ev = p.evict_idx + it.ev0 + it.blk * kTile;
            const int n_rows = min(kTile, it.E - it.blk * kTile);
            const char* src0 = reinterpret_cast<const char*>(p.k_rows) +
                               2 * ((long long)it.tok_begin * p.k_stride_tok + (long long)it.head * p.k_stride_head) + l16 * 16;
#pragma unroll 8
            for (int st = 0; st < kTile / 2; ++st) {
                const int r = 2 * st + (lane >> 4);
                const bool valid = r < n_rows;
                int pos = valid ? __ldg(ev + r) : 0;
                if (pos < 0 || pos >= it.L) { atomicExch(p.status, (int)LOOKM_ERR_DEVICE_BAD_INDEX); pos = 0; }
                const char* src = src0 + 2 * (long long)pos * p.k_stride_tok;
                const uint32_t dst = adst + r * 128 + ((c8 ^ (r & 7)) << 4);
                const int nbytes = valid ? 16 : 0;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(nbytes) : "memory");
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            ptx::fence_proxy_async_shared();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.a_full[ab]));
        }
    } else if (warp == 1 || warp == kEpiWarp0 + kParts * 4) {
        // ------------------------------------------------------------ MMA issuers -----------
        // One thread spends about as long on the waits, fences, commits and loop bookkeeping of a
        // tile as the tensor core needs for its eight MMAs, and it is blocked while they are
        // queued.  Two threads (in warps of different SM sub-partitions) therefore take the tiles
        // alternately: one prepares its next tile while the other one's MMAs run.
        if (lane == 0) {
            const uint32_t me = (warp == 1) ? 0u : 1u;
            constexpr uint32_t idesc = ptx::umma_idesc_bf16(kTile, kTile);
            uint32_t gb = 0;
            int n = 0;
            bool stop = false;                       // a wait gave up: issue nothing more
            for (int round = 0; !stop; ++round, ++n) {
                const int item = item_of_round(round, blockIdx.x, n_cta);
                if (item >= p.n_items) { if (round * n_cta >= p.n_items) break; --n; continue; }
                const Item it = decode_item<KIND>(p, tbl, item);
                const int ab = n % kABuf;
                if (!ptx::mbar_wait(ptx::smem_u32(&sh.a_full[ab]), (n / kABuf) & 1, abort_flag)) break;
                const uint32_t a_addr = ptx::smem_u32(&sh.a[ab][0]);
                bool issued = false;
                for (int t = 0; t < it.nt; ++t, ++gb) {
                    if ((gb & (kIssuers - 1)) != me) continue;
                    const int s = gb % kStages;
                    const int buf = gb % kAccum;
                    // no MMA is issued on operands that have not landed or into an accumulator that
                    // is still being read
                    if (!ptx::mbar_wait(ptx::smem_u32(&sh.b_full[s]), (gb / kStages) & 1, abort_flag) ||
                        !ptx::mbar_wait(ptx::smem_u32(&sh.t_empty[buf]), ((gb / kAccum) & 1) ^ 1, abort_flag)) {
                        stop = true;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t b_addr = ptx::smem_u32(&sh.b[s][0]);
                    const uint32_t d_tmem = tmem_base + buf * kTile;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        // 16 bf16 (32 bytes) per MMA along the 128-byte swizzled row; the second
                        // half of head_dim lives in the second TMA box.
                        const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                        ptx::umma_bf16(d_tmem, ptx::umma_desc_sw128(a_addr + off),
                                       ptx::umma_desc_sw128(b_addr + off), idesc, kk > 0);
                    }
                    if (KIND == kSweep2)                 // accumulator += ones x (-lse / scale)^T
                        ptx::umma_bf16(d_tmem, ptx::umma_desc_sw32(ptx::smem_u32(&sh.ax[0])),
                                       ptx::umma_desc_sw32(ptx::smem_u32(&sh.bx[s % Shared<KIND>::kXStages][0])), idesc, 1u);
                    ptx::umma_commit(ptx::smem_u32(&sh.b_empty[s]));
                    ptx::umma_commit(ptx::smem_u32(&sh.t_full[gb % kFullRing]));
                    issued = true;
                }
                if (stop) break;
                // the stationary tile is free when both issuers are through with the item: an
                // issuer that used it arrives when its MMAs have completed, the other one at once
                if (issued) ptx::umma_commit(ptx::smem_u32(&sh.a_empty[ab]));
                else ptx::mbar_arrive(ptx::smem_u32(&sh.a_empty[ab]));
            }
            // Nothing may release TMEM or leave the kernel while an MMA is still running, also
            // after an abort: wait for all of them (own time limit, the abort flag is ignored).
            int ignore = 0;
            ptx::umma_commit(ptx::smem_u32(&sh.mma_done));
            ptx::mbar_wait(ptx::smem_u32(&sh.mma_done), 0, &ignore, 1000000000ull);
        }
    } else {
        // ------------------------------------------------------------ epilogue --------------
        const int part = (warp - kEpiWarp0) >> 2;            // four-warp unit of the epilogue
        const int wg = part / kHalves;                       // its group
        const int col0 = (part % kHalves) * kCols;           // first accumulator column it reads
        const int quarter = warp & 3;                        // TMEM lane quarter this warp may read
        const int row = quarter * 32 + lane;                 // row of the stationary tile
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const float c2 = p.scale_log2;
        uint32_t gb = 0;
        uint32_t lt = 0;                                     // tiles taken by this group
        int n = 0;
        for (int round = 0;; ++round, ++n) {
            const int item = item_of_round(round, blockIdx.x, n_cta);
            if (item >= p.n_items) { if (round * n_cta >= p.n_items) break; --n; continue; }
            const Item it = decode_item<KIND>(p, tbl, item);
            const int pos = it.blk * kTile + row;            // position of this thread's row (match: its
                                                             // index in the evicted list)
            float m_run = -INFINITY, l_run = 0.f;            // sweep 1
            float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;   // sweep 2
            float best = -INFINITY;                          // match
            int best_slot = 0x7fffffff;
            // match: 1 / |k| of this thread's evicted row takes two dependent loads (its position, then
            // the norm).  They are requested here and after the part's first tile, not in the combine
            // at the item's end, where the part that combines would sit out both round trips while
            // its next accumulator stays full.
            int row_at = 0;
            float row_rnorm = 0.f;
            bool rnorm_asked = false;
            if (KIND == kMatch && pos < it.E) row_at = ptx::ld_nc_s32(p.evict_idx + it.ev0 + pos);
            auto ask_rnorm = [&]() {
                if (pos < it.E) {
                    int at = row_at;
                    if (at < 0 || at >= it.L) at = 0;       // reported by the gather warp
                    row_rnorm = ptx::ld_nc_f32(p.rnorm_all + (long long)it.head * p.T + it.tok_begin + at);
                }
                rnorm_asked = true;
            };

            for (int t = 0; t < it.nt; ++t, ++gb) {
                if ((int)(gb % kGroups) != wg) continue;
                const int buf = (int)(gb % kAccum);
                float* side = sh.side[part][lt & 1];
                bool diag = false;                           // tile crosses the causal diagonal
                int col_limit = kTile;                       // valid columns of the tile (match, sweep 2)
                int diag_from = 0;                           // sweep 2: first column this row may use
                if (KIND == kSweep1) {
                    diag = (t == it.blk);
                } else if (KIND == kSweep2) {
                    const int ib = it.blk + t / p.group;
                    // columns to mask: below the diagonal in the item's first query block, and past
                    // the end of the request in its last one (rows of the next request or zeros)
                    col_limit = min(kTile, it.L - ib * kTile);
                    diag = (ib == it.blk) || (col_limit < kTile);
                    diag_from = (ib == it.blk) ? row : 0;
                } else {
                    if (row < kCols) {
                        const int slot = t * kTile + col0 + row;
                        side[row] = (slot < it.B) ? p.rnorm_kept[it.kept_row0 + slot] : 0.f;
                    }
                    col_limit = min(kTile, it.B - t * kTile);
                    ptx::named_barrier_sync(1 + part, 128);
                }
                ++lt;
                ptx::mbar_wait(ptx::smem_u32(&sh.t_full[gb % kFullRing]), (gb / kFullRing) & 1, abort_flag);
                ptx::tc_fence_after_sync();
                if (KIND == kMatch) {
                    // running arg-max of dot / |kept key| over kept slots, 16 columns at a time with
                    // the next 16 already on their way from TMEM (a load takes about as long as
                    // the work on 32 columns).  The maximum of the 16 is taken first; only when it
                    // beats the running best is its first column looked up, so a strict comparison
                    // in ascending slot order keeps the lowest slot.
                    auto columns16 = [&](const uint32_t (&r)[16], int c0) {      // c0: column of the tile
                        const float4* sd = reinterpret_cast<const float4*>(side + (c0 - col0));
                        float v[16];
#pragma unroll
                        for (int c4 = 0; c4 < 4; ++c4) {
                            const float4 r4 = sd[c4];
                            v[c4 * 4 + 0] = __uint_as_float(r[c4 * 4 + 0]) * r4.x;
                            v[c4 * 4 + 1] = __uint_as_float(r[c4 * 4 + 1]) * r4.y;
                            v[c4 * 4 + 2] = __uint_as_float(r[c4 * 4 + 2]) * r4.z;
                            v[c4 * 4 + 3] = __uint_as_float(r[c4 * 4 + 3]) * r4.w;
                        }
                        if (col_limit < kTile) {           // last tile of the kept list only
#pragma unroll
                            for (int c = 0; c < 16; ++c)
                                if (c0 + c >= col_limit) v[c] = -INFINITY;
                        }
                        const float m0 = ptx::fmax3(v[0], v[1], v[2]);
                        const float m1 = ptx::fmax3(v[3], v[4], v[5]);
                        const float m2 = ptx::fmax3(v[6], v[7], v[8]);
                        const float m3 = ptx::fmax3(v[9], v[10], v[11]);
                        const float m4 = ptx::fmax3(v[12], v[13], v[14]);
                        const float mx = fmaxf(ptx::fmax3(m0, m1, m2), ptx::fmax3(m3, m4, v[15]));
                        if (mx > best) {
                            best = mx;
                            int idx = 15;
#pragma unroll
                            for (int c = 14; c >= 0; --c) if (v[c] == mx) idx = c;
                            best_slot = t * kTile + c0 + idx;
                        }
                    };
                    uint32_t ra[16], rb[16];
                    const uint32_t tbase = lane_addr + buf * kTile + col0;
                    ptx::tmem_ld_32x16(tbase, ra);
#pragma unroll
                    for (int k = 0; k < kCols / 32; ++k) {
                        ptx::tmem_ld_wait16(ra);
                        ptx::tmem_ld_32x16(tbase + (2 * k + 1) * 16, rb, ra);
                        columns16(ra, col0 + 2 * k * 16);
                        ptx::tmem_ld_wait16(rb);
                        if (k < kCols / 32 - 1) {
                            ptx::tmem_ld_32x16(tbase + (2 * k + 2) * 16, ra, rb);
                        } else {
                            // everything is in registers: hand the accumulator back
                            ptx::tc_fence_before_sync();
                            __syncwarp();
                            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.t_empty[buf]));
                        }
                        columns16(rb, col0 + (2 * k + 1) * 16);
                    }
                    if (!rnorm_asked) ask_rnorm();
                    continue;
                }
                // work on 32 columns of the accumulator, c0 = first column of the chunk
                auto process = [&](const uint32_t (&raw)[32], int c0) {
                    if (KIND == kSweep1) {
                        // softmax statistics of row `pos` over key columns c0..c0+31: l_run is the
                        // sum of exp2(x - m_run), where m_run is a REFERENCE, not necessarily the
                        // maximum so far
                        if (diag) {
                            // diagonal tile (the last of the item): exact running maximum
                            float mx = m_run;
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (c0 + c <= row) mx = fmaxf(mx, __uint_as_float(raw[c]));
                            if (mx != -INFINITY) {           // false only above the diagonal
                                const float mc = mx * c2;
                                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                                for (int c = 0; c < 32; c += 2) {
                                    const float e0 = exp2_mixed(c, fmaf(__uint_as_float(raw[c]), c2, -mc));
                                    const float e1 = exp2_mixed(c + 1, fmaf(__uint_as_float(raw[c + 1]), c2, -mc));
                                    s0 += (c0 + c <= row) ? e0 : 0.f;
                                    s1 += (c0 + c + 1 <= row) ? e1 : 0.f;
                                }
                                l_run = l_run * ptx::ex2(m_run * c2 - mc) + (s0 + s1);
                                m_run = mx;
                            }
                        } else {
                            // Full tiles: no maximum is taken.  The reference is the maximum of the
                            // row's first 32 columns; later logits may exceed it as long as the
                            // chunk's sum stays below 2^60 (fp32 has the range, and the relative
                            // precision does not depend on the reference).  When it does not, or
                            // overflows, the chunk is redone against its true maximum.
                            float ref = m_run;           // -inf at the row's first chunk: the sum
                            float sum;                   // overflows and the second round sets it
#pragma unroll 1
                            for (int round2 = 0;; ++round2) {
                                const float mc = ref * c2;
                                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                                for (int c = 0; c < 32; c += 2) {
                                    s0 += exp2_mixed(c, fmaf(__uint_as_float(raw[c]), c2, -mc));
                                    s1 += exp2_mixed(c + 1, fmaf(__uint_as_float(raw[c + 1]), c2, -mc));
                                }
                                sum = s0 + s1;
                                if (sum < kReferenceSlack || round2) break;
                                float mx = ref;
#pragma unroll
                                for (int c = 0; c < 32; c += 2)
                                    mx = ptx::fmax3(mx, __uint_as_float(raw[c]), __uint_as_float(raw[c + 1]));
                                l_run *= ptx::ex2(ref * c2 - mx * c2);
                                ref = mx;
                            }
                            l_run += sum;
                            m_run = ref;
                        }
                    } else if (KIND == kSweep2) {
                        // probabilities of key `pos` under query columns c0..c0+31: the accumulator
                        // holds s_ij - lse_i / scale
                        if (diag) {
#pragma unroll
                            for (int c4 = 0; c4 < 8; ++c4) {
                                const int c = c0 + c4 * 4;
                                const float e0 = exp2_mixed(c4 * 4 + 0, __uint_as_float(raw[c4 * 4 + 0]) * c2);
                                const float e1 = exp2_mixed(c4 * 4 + 1, __uint_as_float(raw[c4 * 4 + 1]) * c2);
                                const float e2 = exp2_mixed(c4 * 4 + 2, __uint_as_float(raw[c4 * 4 + 2]) * c2);
                                const float e3 = exp2_mixed(c4 * 4 + 3, __uint_as_float(raw[c4 * 4 + 3]) * c2);
                                acc0 += (c + 0 >= diag_from && c + 0 < col_limit) ? e0 : 0.f;
                                acc1 += (c + 1 >= diag_from && c + 1 < col_limit) ? e1 : 0.f;
                                acc2 += (c + 2 >= diag_from && c + 2 < col_limit) ? e2 : 0.f;
                                acc3 += (c + 3 >= diag_from && c + 3 < col_limit) ? e3 : 0.f;
                            }
                        } else {
#pragma unroll
                            for (int c4 = 0; c4 < 8; ++c4) {
                                acc0 += exp2_mixed(c4 * 4 + 0, __uint_as_float(raw[c4 * 4 + 0]) * c2);
                                acc1 += exp2_mixed(c4 * 4 + 1, __uint_as_float(raw[c4 * 4 + 1]) * c2);
                                acc2 += exp2_mixed(c4 * 4 + 2, __uint_as_float(raw[c4 * 4 + 2]) * c2);
                                acc3 += exp2_mixed(c4 * 4 + 3, __uint_as_float(raw[c4 * 4 + 3]) * c2);
                            }
                        }
                    }
                };
                // the last columns are in registers: hand the accumulator back, so that the next
                // tile's MMAs run while this chunk is still being worked on
                auto release = [&]() {
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.t_empty[buf]));
                };
                const uint32_t tbase = lane_addr + buf * kTile + col0;
#pragma unroll 1
                for (int ch = 0; ch < kCols / 32; ++ch) {
                    uint32_t raw[32];
                    ptx::tmem_ld_32x32(tbase + ch * 32, raw);
                    ptx::tmem_ld_wait();
                    if (ch == kCols / 32 - 1) release();
                    process(raw, col0 + ch * 32);
                }
            }

            // ---- combine the four groups and write this item's results -----------------------
            // The group that owns the item's last tile finishes last anyway, so it combines: the
            // others leave their partial results in shared memory, signal, and go on to the next
            // item without waiting for anybody.  Values are always combined in group order.
            const int cslot = n & 1;
            const uint32_t cuse = static_cast<uint32_t>(n) >> 1;         // earlier uses of this buffer
            const int combiner = static_cast<int>((gb - 1u) % kGroups) * kHalves + (kHalves - 1);
            float (*cb)[Shared<KIND>::kPlanes][kTile] = sh.comb[cslot];
            constexpr int kP1 = Shared<KIND>::kPlanes - 1;       // second value of a row (not in sweep 2)
            if (part != combiner) {
                // the buffer's previous contents (two items ago) have been read
                ptx::mbar_wait(ptx::smem_u32(&sh.comb_free[cslot]), (cuse & 1u) ^ 1u, abort_flag);
                if (KIND == kSweep1) { cb[part][0][row] = m_run; cb[part][kP1][row] = l_run; }
                else if (KIND == kSweep2) { cb[part][0][row] = (acc0 + acc1) + (acc2 + acc3); }
                else { cb[part][0][row] = best; cb[part][kP1][row] = __int_as_float(best_slot); }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.comb_full[cslot]));
            } else {
                ptx::mbar_wait(ptx::smem_u32(&sh.comb_full[cslot]), cuse & 1u, abort_flag);
                if (pos < (KIND == kMatch ? it.E : it.L) && !*abort_flag) {
                    if (KIND == kSweep1) {
                        float mg[kParts], lg[kParts];
#pragma unroll
                        for (int g = 0; g < kParts; ++g) {
                            mg[g] = (g == part) ? m_run : cb[g][0][row];
                            lg[g] = (g == part) ? l_run : cb[g][kP1][row];
                        }
                        float m = mg[0];
#pragma unroll
                        for (int g = 1; g < kParts; ++g) m = fmaxf(m, mg[g]);
                        float l = lg[0] * ptx::ex2((mg[0] - m) * c2);
#pragma unroll
                        for (int g = 1; g < kParts; ++g) l += lg[g] * ptx::ex2((mg[g] - m) * c2);
                        // natural-log log-sum-exp of the scaled logits
                        const float lse = (m * c2 + ptx::lg2(l)) * kLn2;
                        p.lse[(long long)it.head * p.T + it.tok_begin + pos] = lse;
                        store_lse_split(p.lse_split + ((long long)(it.tok_begin + pos) * p.n_q_heads + it.head) * 16,
                                        lse, c2);
                    } else if (KIND == kSweep2) {
                        const float own = (acc0 + acc1) + (acc2 + acc3);
                        float a = (part == 0) ? own : cb[0][0][row];
#pragma unroll
                        for (int g = 1; g < kParts; ++g) a += (g == part) ? own : cb[g][0][row];
                        p.scores[(long long)it.head * p.T + it.tok_begin + pos] = a;
                    } else {
                        if (!rnorm_asked) ask_rnorm();           // a part without a tile in this item
                        const int e = pos;
                        {
                            float bb = (part == 0) ? best : cb[0][0][row];
                            int bs = (part == 0) ? best_slot : __float_as_int(cb[0][kP1][row]);
#pragma unroll
                            for (int g = 1; g < kParts; ++g) {
                                const float b1 = (g == part) ? best : cb[g][0][row];
                                const int s1 = (g == part) ? best_slot : __float_as_int(cb[g][kP1][row]);
                                if (b1 > bb || (b1 == bb && s1 < bs)) { bb = b1; bs = s1; }
                            }
                            p.assign[it.ev0 + e] = bs;
                            p.sim[it.ev0 + e] = bb * row_rnorm;
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.comb_free[cslot]));
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && sh.abort_flag) atomicExch(p.status, (int)LOOKM_ERR_DEVICE_TIMEOUT);
}

// The failure path of the bounded waits, exercised without starving a production kernel: thread 0
// waits with ptx::mbar_wait on an mbarrier that nobody arrives at, the other threads on the same
// barrier see either the limit or the abort flag, and the CTA reports the expiry exactly as
// tile_kernel does (shared abort flag -> status word).
__global__ void __launch_bounds__(128)
wait_probe_kernel(unsigned long long limit_ns, int* status) {
    __shared__ unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&bar), 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    volatile int* flag = &abort_flag;
    const bool arrived = ptx::mbar_wait(ptx::smem_u32(&bar), 0, flag, limit_ns);
    __syncthreads();
    if (threadIdx.x == 0 && (abort_flag || !arrived)) atomicExch(status, (int)LOOKM_ERR_DEVICE_TIMEOUT);
}

}  // namespace

cudaError_t launch_wait_probe(unsigned long long limit_ns, int* status, cudaStream_t stream) {
    wait_probe_kernel<<<1, 128, 0, stream>>>(limit_ns, status);
    return cudaGetLastError();
}

cudaError_t launch_tile_kernel(int kind, const CUtensorMap& map_a, const CUtensorMap& map_b,
                               const CUtensorMap* map_x, const TileParams& p, int num_sms,
                               cudaStream_t stream) {
    if (p.n_items <= 0) return cudaSuccess;
    const int smem_of[3] = {(int)sizeof(Shared<kSweep1>) + 1024, (int)sizeof(Shared<kSweep2>) + 1024,
                            (int)sizeof(Shared<kMatch>) + 1024};
    const int grid = p.n_items < num_sms ? p.n_items : num_sms;
    const CUtensorMap& mx = map_x ? *map_x : map_b;      // only sweep 2 uses it
    static unsigned long long configured = 0;
    cudaError_t err = once_per_device(configured, [&]() {
        cudaError_t e = cudaFuncSetAttribute(tile_kernel<kSweep1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_of[kSweep1]);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(tile_kernel<kSweep2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_of[kSweep2]);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(tile_kernel<kMatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_of[kMatch]);
        return e;
    });
    if (err != cudaSuccess) return err;
    if (kind == kSweep1)
        return launch_chained(tile_kernel<kSweep1>, dim3(grid), dim3(threads_of(kSweep1)), (size_t)smem_of[kSweep1], stream, map_a, map_b, mx, p);
    if (kind == kSweep2)
        return launch_chained(tile_kernel<kSweep2>, dim3(grid), dim3(threads_of(kSweep2)), (size_t)smem_of[kSweep2], stream, map_a, map_b, mx, p);
    return launch_chained(tile_kernel<kMatch>, dim3(grid), dim3(threads_of(kMatch)), (size_t)smem_of[kMatch], stream, map_a, map_b, mx, p);
}

cudaError_t launch_lse_split(const float* lse, int n_q_heads, long long T, float scale_log2,
                             unsigned short* lse_split, cudaStream_t stream) {
    const long long n = T * n_q_heads;
    if (n <= 0) return cudaSuccess;
    lse_split_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(lse, n_q_heads, T, scale_log2, lse_split);
    return cudaGetLastError();
}

}  // namespace lookm
