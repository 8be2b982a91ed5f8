// Tensor-core kernels of the path: the two sweeps of the cumulative attention score (Eq. 4) and
// the cosine matching with fused row argmax (Eq. 9).
//
// All three are the same persistent, warp-specialised pipeline over 128 x 128 x 128 bf16 tiles:
//   - a work item owns TWO stationary 128-row tiles (256 consecutive rows of the A operand; the
//     rows of each tile sit on the 128 TMEM lanes) and streams a sequence of 128-row tiles (the B
//     operand) against them, so every streamed tile feeds two MMAs (16 tcgen05.mma of
//     128 x 128 x 16) and the L2 -> shared-memory traffic per flop is halved;
//   - warp 0 (one thread) issues the TMA loads; warps 1 and 18 (one thread each) issue the MMAs
//     of the even and of the odd streamed tiles into four 128-column TMEM accumulators (streamed
//     tile parity x stationary tile).  Measured on B200: a thread that waits on an mbarrier,
//     fences and commits between every 8 MMAs keeps the tensor pipe only about half busy (512
//     clocks per 8 MMAs alone, about 900 with one wait and two commits in between), so the
//     synchronisation is done once per streamed tile and two threads alternate;
//   - two groups of four warps run the epilogue, one group per stationary tile, alternating
//     between that tile's two accumulators (so the MMA of the next streamed tile runs meanwhile).
//     A thread reads its whole accumulator row (128 columns, four tcgen05.ld.x32 in flight, one
//     wait) before it computes: the TMEM load latency of several hundred clocks is then paid once
//     per tile, which is what lets two warps per SM sub-partition keep the exp unit busy;
//   - each epilogue thread owns one row of its stationary tile for the whole item, so every
//     reduction over the streamed axis (row maximum and sum, column-sum of probabilities for one
//     key, running arg-max) stays in that thread's registers.  No L x L matrix is ever stored.
//
//   sweep 1: A = 256 queries of one query head, B = key tiles 0..diagonal.  Online softmax
//            statistics per query row  ->  lse[i] = log sum_{j<=i} exp(s_ij).
//   sweep 2: A = 256 keys of one KV head, B = query tiles diagonal..last of every query head in
//            the group.  Thread of key j accumulates sum_i exp(s_ij - lse_i)  ->  A_s[j].
//   match  : A = 256 key rows (all positions; kept rows are ignored at the end), B = tiles of the
//            compacted kept keys.  Thread keeps the largest s_ij / |k_j| and its slot.
//
// Work items are laid out heaviest first and dealt to the CTAs in serpentine order; every role
// walks the same item sequence on its own, so no scheduling state is shared.
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace lookm {
namespace {

constexpr int kStages = 4;                       // ring of streamed tiles
constexpr int kGroups = 2;                       // epilogue groups (one per stationary tile)
constexpr int kMmaWarp1 = 2 + kGroups * 4;       // the second MMA-issuing warp
constexpr int kThreads = (kMmaWarp1 + 1) * 32;   // producer, MMA (even), 2 x 4 epilogue, MMA (odd)
constexpr int kHalfBytes = kTile * 64 * 2;       // one TMA box: 128 rows x 64 bf16 (128 B rows)
constexpr int kTileBytes = 2 * kHalfBytes;       // 128 x 128 bf16
constexpr int kReqCache = 32;                    // request-table entries cached in shared memory
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct __align__(1024) Shared {
    uint8_t a[2][kTileBytes];                    // the item's two stationary tiles
    uint8_t b[kStages][kTileBytes];              // streamed tiles
    alignas(16) float side[kGroups][2][kTile];   // per epilogue group, double-buffered column data
    Req reqs[kReqCache];
    unsigned long long a_full, a_empty;
    unsigned long long b_full[kStages], b_empty[kStages];
    unsigned long long t_full[2], t_empty[2];    // per streamed-tile parity (two accumulators each)
    unsigned long long mma_done;                 // every MMA of this CTA has completed
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Shared) + 1024 <= 232448, "shared storage exceeds what one CTA may use");

struct Item {
    int tok_begin, L, B, bp, head, nt, nblk;
    long long kept_row0;      // match: first row of this (request, head) in the kept-key matrix
    long long ev0;            // match: start of its evicted list
};

// Work item `item` of stage KIND.  An item covers block pair bp = stationary blocks 2bp, 2bp+1.
template <int KIND>
__device__ __forceinline__ Item decode_item(const TileParams& p, const Req* tbl, int item) {
    int lo = 0, hi = p.n_req - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (tbl[mid].item_begin[KIND] <= item) lo = mid; else hi = mid - 1;
    }
    const Req& rq = tbl[lo];
    const int u = item - rq.item_begin[KIND];
    const int npair = (rq.nblk + 1) >> 1;
    Item it;
    it.tok_begin = rq.tok_begin;
    it.L = rq.L;
    it.B = rq.B;
    it.nblk = rq.nblk;
    it.kept_row0 = 0;
    it.ev0 = 0;
    if (KIND == kSweep1) {                       // heaviest first: last query blocks first
        it.bp = npair - 1 - u / p.n_q_heads;
        it.head = u % p.n_q_heads;
        it.nt = min(rq.nblk, 2 * it.bp + 2);     // key tiles 0 .. the later block's diagonal
    } else if (KIND == kSweep2) {                // heaviest first: first key blocks first
        it.bp = u / p.n_kv_heads;
        it.head = u % p.n_kv_heads;
        it.nt = (rq.nblk - 2 * it.bp) * p.group;
    } else {
        it.bp = u / p.n_kv_heads;
        it.head = u % p.n_kv_heads;
        it.nt = (rq.B + kTile - 1) / kTile;
        it.kept_row0 = rq.kept_off + (long long)it.head * rq.B;
        it.ev0 = rq.ev_off + (long long)it.head * rq.E;
    }
    return it;
}

// Does streamed tile t contribute anything to stationary tile `sub` of the item?  (The block may
// lie past the prompt end, or the whole tile may be on the wrong side of the causal diagonal.)
template <int KIND>
__device__ __forceinline__ bool unit_active(const TileParams& p, const Item& it, int t, int sub) {
    const int blk = 2 * it.bp + sub;
    if (blk >= it.nblk) return false;
    if (KIND == kSweep1) return t <= blk;                          // keys up to the query block
    if (KIND == kSweep2) return 2 * it.bp + t / p.group >= blk;    // queries from the key block on
    return true;
}

// Serpentine deal of the item list: round k hands items k*G .. k*G+G-1 to the CTAs in forward
// order when k is even and in reverse order when k is odd.
__device__ __forceinline__ int item_of_round(int round, int cta, int n_cta) {
    return round * n_cta + ((round & 1) ? (n_cta - 1 - cta) : cta);
}

template <int KIND>
__global__ void __launch_bounds__(kThreads, 1)
tile_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const TileParams p) {
    extern __shared__ uint8_t smem_raw[];
    Shared& sh = *reinterpret_cast<Shared*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    volatile int* abort_flag = &sh.abort_flag;

    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&sh.a_full), 1);
        ptx::mbar_init(ptx::smem_u32(&sh.a_empty), 2);         // one arrival per MMA thread
        for (int i = 0; i < kStages; ++i) {
            ptx::mbar_init(ptx::smem_u32(&sh.b_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.b_empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(ptx::smem_u32(&sh.t_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.t_empty[i]), 8);  // one arrival per warp of two groups
        }
        ptx::mbar_init(ptx::smem_u32(&sh.mma_done), 2);
        sh.abort_flag = 0;
        ptx::fence_mbar_init();
    }
    const Req* tbl = p.reqs;
    if (p.n_req <= kReqCache) {                  // the table is read once per item by every role
        for (int i = threadIdx.x; i < p.n_req * (int)(sizeof(Req) / 4); i += kThreads)
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
            uint32_t gb = 0;                         // running streamed-tile index
            int n = 0;                               // items done by this CTA
            for (int round = 0;; ++round, ++n) {
                const int item = item_of_round(round, blockIdx.x, n_cta);
                if (item >= p.n_items) { if (round * n_cta >= p.n_items) break; --n; continue; }
                const Item it = decode_item<KIND>(p, tbl, item);
                // both stationary tiles; rows past the tensor end read as zero
                ptx::mbar_wait(ptx::smem_u32(&sh.a_empty), (n & 1) ^ 1, abort_flag);
                const uint32_t abar = ptx::smem_u32(&sh.a_full);
                ptx::mbar_arrive_expect_tx(abar, 2 * kTileBytes);
#pragma unroll
                for (int sub = 0; sub < 2; ++sub) {
                    const uint32_t adst = ptx::smem_u32(&sh.a[sub][0]);
                    const int a_row = it.tok_begin + (2 * it.bp + sub) * kTile;
                    ptx::tma_load_3d(adst, &map_a, 0, it.head, a_row, abar);
                    ptx::tma_load_3d(adst + kHalfBytes, &map_a, 64, it.head, a_row, abar);
                }
                for (int t = 0; t < it.nt; ++t, ++gb) {
                    const int s = gb % kStages;
                    ptx::mbar_wait(ptx::smem_u32(&sh.b_empty[s]), ((gb / kStages) & 1) ^ 1, abort_flag);
                    const uint32_t bbar = ptx::smem_u32(&sh.b_full[s]);
                    ptx::mbar_arrive_expect_tx(bbar, kTileBytes);
                    const uint32_t bdst = ptx::smem_u32(&sh.b[s][0]);
                    if (KIND == kSweep1) {
                        const int row = it.tok_begin + t * kTile;
                        const int h = it.head / p.group;
                        ptx::tma_load_3d(bdst, &map_b, 0, h, row, bbar);
                        ptx::tma_load_3d(bdst + kHalfBytes, &map_b, 64, h, row, bbar);
                    } else if (KIND == kSweep2) {
                        const int row = it.tok_begin + (2 * it.bp + t / p.group) * kTile;
                        const int h = it.head * p.group + t % p.group;
                        ptx::tma_load_3d(bdst, &map_b, 0, h, row, bbar);
                        ptx::tma_load_3d(bdst + kHalfBytes, &map_b, 64, h, row, bbar);
                    } else {
                        const int row = (int)(it.kept_row0 + (long long)t * kTile);
                        ptx::tma_load_2d(bdst, &map_b, 0, row, bbar);
                        ptx::tma_load_2d(bdst + kHalfBytes, &map_b, 64, row, bbar);
                    }
                }
            }
            // Every load issued above is consumed by an MMA thread before it finishes, except
            // after an abort: then wait (bounded, ignoring the flag) until the last ring of
            // loads has landed so that no copy is in flight when the CTA exits.
            if (*abort_flag) {
                int dummy = 0;
                const uint32_t last = gb;
                for (uint32_t g = (last > (uint32_t)kStages ? last - kStages : 0); g < last; ++g)
                    ptx::mbar_wait(ptx::smem_u32(&sh.b_full[g % kStages]), (g / kStages) & 1, &dummy,
                                   200000000ull);
            }
        }
    } else if (warp == 1 || warp == kMmaWarp1) {
        // ------------------------------------------------------------ MMA issuers -----------
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::umma_idesc_bf16(kTile, kTile);
            const uint32_t mine = (warp == 1) ? 0u : 1u;     // parity of the streamed tiles I issue
            uint32_t gb = 0;
            int n = 0;
            for (int round = 0;; ++round, ++n) {
                const int item = item_of_round(round, blockIdx.x, n_cta);
                if (item >= p.n_items) { if (round * n_cta >= p.n_items) break; --n; continue; }
                const Item it = decode_item<KIND>(p, tbl, item);
                // my last streamed tile of this item (-1: its only tile has the other parity)
                int last_t = it.nt - 1;
                if (((gb + last_t) & 1u) != mine) --last_t;
                // Always wait for this item's stationary tiles: their arrival also proves that the
                // previous item's a_empty phase is over, so the arrival below cannot fall into it.
                ptx::mbar_wait(ptx::smem_u32(&sh.a_full), n & 1, abort_flag);
                if (last_t < 0) ptx::mbar_arrive(ptx::smem_u32(&sh.a_empty));
                for (int t = 0; t < it.nt; ++t, ++gb) {
                    if ((gb & 1u) != mine) continue;
                    const int s = gb % kStages;
                    ptx::mbar_wait(ptx::smem_u32(&sh.b_full[s]), (gb / kStages) & 1, abort_flag);
                    ptx::mbar_wait(ptx::smem_u32(&sh.t_empty[mine]), ((gb >> 1) & 1) ^ 1, abort_flag);
                    ptx::tc_fence_after_sync();
                    const uint32_t b_addr = ptx::smem_u32(&sh.b[s][0]);
#pragma unroll
                    for (int sub = 0; sub < 2; ++sub) {
                        if (unit_active<KIND>(p, it, t, sub)) {
                            const uint32_t a_addr = ptx::smem_u32(&sh.a[sub][0]);
                            const uint32_t d_tmem = tmem_base + (2 * mine + sub) * kTile;
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk) {
                                // 16 bf16 (32 bytes) per MMA along the 128-byte swizzled row; the
                                // second half of head_dim lives in the second TMA box.
                                const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                                ptx::umma_bf16(d_tmem, ptx::umma_desc_sw128(a_addr + off),
                                               ptx::umma_desc_sw128(b_addr + off), idesc, kk > 0);
                            }
                        }
                    }
                    ptx::umma_commit(ptx::smem_u32(&sh.t_full[mine]));
                    ptx::umma_commit(ptx::smem_u32(&sh.b_empty[s]));
                    if (t == last_t) ptx::umma_commit(ptx::smem_u32(&sh.a_empty));
                }
            }
            // Nothing may release TMEM or leave the kernel while an MMA is still running, also
            // after an abort: wait for all of them (own time limit, the abort flag is ignored).
            int ignore = 0;
            ptx::umma_commit(ptx::smem_u32(&sh.mma_done));
            ptx::mbar_wait(ptx::smem_u32(&sh.mma_done), 0, &ignore, 1000000000ull);
        }
    } else {
        // ------------------------------------------------------------ epilogue --------------
        const int sub = (warp - 2) >> 2;                     // epilogue group = stationary tile
        const int quarter = warp & 3;                        // TMEM lane quarter this warp may read
        const int row = quarter * 32 + lane;                 // row of the stationary tile
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const float c2 = p.scale_log2;
        uint32_t gb = 0;
        uint32_t lt = 0;                                     // staged tiles of this group
        for (int round = 0;; ++round) {
            const int item = item_of_round(round, blockIdx.x, n_cta);
            if (item >= p.n_items) { if (round * n_cta >= p.n_items) break; continue; }
            const Item it = decode_item<KIND>(p, tbl, item);
            const int blk = 2 * it.bp + sub;                 // this group's stationary block
            const int pos = blk * kTile + row;               // position of this thread's row
            float m_run = -INFINITY, l_run = 0.f;            // sweep 1
            float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;   // sweep 2
            float best = -INFINITY;                          // match
            int best_slot = 0x7fffffff;

            // per-column data of streamed tile t, for the column this thread stages:
            // sweep 2: log2-sum-exp of the query (+inf past the prompt end: probability 0);
            // match  : inverse norm of the kept key (0 past the last kept slot)
            auto side_value = [&](int t) -> float {
                if (KIND == kSweep2) {
                    const int i = (2 * it.bp + t / p.group) * kTile + row;
                    const int qh = it.head * p.group + t % p.group;
                    return (i < it.L) ? p.lse[(long long)qh * p.T + it.tok_begin + i] * kLog2e : INFINITY;
                } else if (KIND == kMatch) {
                    const int slot = t * kTile + row;
                    return (slot < it.B) ? p.rnorm_kept[it.kept_row0 + slot] : 0.f;
                }
                return 0.f;
            };
            // first active tile of this group, so that its column data can be fetched ahead
            int t_next = 0;
            while (t_next < it.nt && !unit_active<KIND>(p, it, t_next, sub)) ++t_next;
            float side_next = (KIND != kSweep1 && t_next < it.nt) ? side_value(t_next) : 0.f;

            for (int t = 0; t < it.nt; ++t, ++gb) {
                const int par = gb & 1;
                const int acc = 2 * par + sub;
                const bool active = unit_active<KIND>(p, it, t, sub);
                float* side = sh.side[sub][lt & 1];
                if (KIND != kSweep1 && active) {
                    side[row] = side_next;                   // fetched during the previous tile
                    ptx::named_barrier_sync(1 + sub, 128);
                    ++lt;
                    t_next = t + 1;                          // later tiles of an item are all active
                    if (t_next < it.nt) side_next = side_value(t_next);
                }
                ptx::mbar_wait(ptx::smem_u32(&sh.t_full[par]), (gb >> 1) & 1, abort_flag);
                ptx::tc_fence_after_sync();
                if (active) {
                    uint32_t raw[kTile];
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch)
                        ptx::tmem_ld_32x32(lane_addr + acc * kTile + ch * 32,
                                           *reinterpret_cast<uint32_t(*)[32]>(&raw[ch * 32]));
                    ptx::tmem_ld_wait128(raw);
                    if (KIND == kSweep1) {
                        // online softmax statistics of row `pos` over the tile's 128 key columns
                        const bool diag = (t == blk);        // keys j <= i only
                        float m0 = m_run, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
                        for (int c = 0; c < kTile; c += 4) {
                            if (!diag || c + 0 <= row) m0 = fmaxf(m0, __uint_as_float(raw[c + 0]));
                            if (!diag || c + 1 <= row) m1 = fmaxf(m1, __uint_as_float(raw[c + 1]));
                            if (!diag || c + 2 <= row) m2 = fmaxf(m2, __uint_as_float(raw[c + 2]));
                            if (!diag || c + 3 <= row) m3 = fmaxf(m3, __uint_as_float(raw[c + 3]));
                        }
                        const float mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));   // finite: column 0 is valid
                        const float mc = mx * c2;
                        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
                        if (diag) {
#pragma unroll
                            for (int c = 0; c < kTile; c += 4) {
                                const float e0 = ptx::ex2(fmaf(__uint_as_float(raw[c + 0]), c2, -mc));
                                const float e1 = ptx::ex2(fmaf(__uint_as_float(raw[c + 1]), c2, -mc));
                                const float e2 = ptx::ex2(fmaf(__uint_as_float(raw[c + 2]), c2, -mc));
                                const float e3 = ptx::ex2(fmaf(__uint_as_float(raw[c + 3]), c2, -mc));
                                s0 += (c + 0 <= row) ? e0 : 0.f;
                                s1 += (c + 1 <= row) ? e1 : 0.f;
                                s2 += (c + 2 <= row) ? e2 : 0.f;
                                s3 += (c + 3 <= row) ? e3 : 0.f;
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < kTile; c += 4) {
                                s0 += ptx::ex2(fmaf(__uint_as_float(raw[c + 0]), c2, -mc));
                                s1 += ptx::ex2(fmaf(__uint_as_float(raw[c + 1]), c2, -mc));
                                s2 += ptx::ex2(fmaf(__uint_as_float(raw[c + 2]), c2, -mc));
                                s3 += ptx::ex2(fmaf(__uint_as_float(raw[c + 3]), c2, -mc));
                            }
                        }
                        l_run = l_run * ptx::ex2(m_run * c2 - mc) + ((s0 + s1) + (s2 + s3));
                        m_run = mx;
                    } else if (KIND == kSweep2) {
                        // probabilities of key `pos` under the tile's 128 query columns
                        const bool diag = (2 * it.bp + t / p.group == blk);   // queries i >= j only
                        const float4* sd = reinterpret_cast<const float4*>(side);
                        if (diag) {
#pragma unroll
                            for (int c4 = 0; c4 < kTile / 4; ++c4) {
                                const float4 l4 = sd[c4];
                                const int c = c4 * 4;
                                const float e0 = ptx::ex2(fmaf(__uint_as_float(raw[c + 0]), c2, -l4.x));
                                const float e1 = ptx::ex2(fmaf(__uint_as_float(raw[c + 1]), c2, -l4.y));
                                const float e2 = ptx::ex2(fmaf(__uint_as_float(raw[c + 2]), c2, -l4.z));
                                const float e3 = ptx::ex2(fmaf(__uint_as_float(raw[c + 3]), c2, -l4.w));
                                acc0 += (c + 0 >= row) ? e0 : 0.f;
                                acc1 += (c + 1 >= row) ? e1 : 0.f;
                                acc2 += (c + 2 >= row) ? e2 : 0.f;
                                acc3 += (c + 3 >= row) ? e3 : 0.f;
                            }
                        } else {
#pragma unroll
                            for (int c4 = 0; c4 < kTile / 4; ++c4) {
                                const float4 l4 = sd[c4];
                                const int c = c4 * 4;
                                acc0 += ptx::ex2(fmaf(__uint_as_float(raw[c + 0]), c2, -l4.x));
                                acc1 += ptx::ex2(fmaf(__uint_as_float(raw[c + 1]), c2, -l4.y));
                                acc2 += ptx::ex2(fmaf(__uint_as_float(raw[c + 2]), c2, -l4.z));
                                acc3 += ptx::ex2(fmaf(__uint_as_float(raw[c + 3]), c2, -l4.w));
                            }
                        }
                    } else {
                        // running arg-max of dot / |kept key| over kept slots: per 16 columns the
                        // maximum first; only a new maximum is searched for its (lowest) column
                        const int col_limit = it.B - t * kTile;      // valid kept slots in the tile
                        const float4* sd = reinterpret_cast<const float4*>(side);
#pragma unroll
                        for (int g16 = 0; g16 < kTile / 16; ++g16) {
                            float v[16];
#pragma unroll
                            for (int c4 = 0; c4 < 4; ++c4) {
                                const float4 r4 = sd[g16 * 4 + c4];
                                const int c = g16 * 16 + c4 * 4;
                                v[c4 * 4 + 0] = __uint_as_float(raw[c + 0]) * r4.x;
                                v[c4 * 4 + 1] = __uint_as_float(raw[c + 1]) * r4.y;
                                v[c4 * 4 + 2] = __uint_as_float(raw[c + 2]) * r4.z;
                                v[c4 * 4 + 3] = __uint_as_float(raw[c + 3]) * r4.w;
                            }
                            if (col_limit < kTile) {
#pragma unroll
                                for (int c = 0; c < 16; ++c) if (g16 * 16 + c >= col_limit) v[c] = -INFINITY;
                            }
                            float mx = v[0];
#pragma unroll
                            for (int c = 1; c < 16; ++c) mx = fmaxf(mx, v[c]);
                            if (mx > best) {                  // strict: an equal value keeps the lower slot
                                best = mx;
                                int idx = 15;
#pragma unroll
                                for (int c = 14; c >= 0; --c) if (v[c] == mx) idx = c;
                                best_slot = t * kTile + g16 * 16 + idx;
                            }
                        }
                    }
                }
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.t_empty[par]));
            }

            // ---- this thread's row is complete: write the item's result --------------------------
            if (pos < it.L && !*abort_flag) {
                if (KIND == kSweep1) {
                    // natural-log log-sum-exp of the scaled logits
                    p.lse[(long long)it.head * p.T + it.tok_begin + pos] = (m_run * c2 + ptx::lg2(l_run)) * kLn2;
                } else if (KIND == kSweep2) {
                    p.scores[(long long)it.head * p.T + it.tok_begin + pos] = (acc0 + acc1) + (acc2 + acc3);
                } else {
                    const long long g = (long long)it.head * p.T + it.tok_begin + pos;
                    const int e = p.rank[g];
                    if (e >= 0) {
                        p.assign[it.ev0 + e] = best_slot;
                        p.sim[it.ev0 + e] = best * p.rnorm_all[g];
                    }
                }
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

}  // namespace

cudaError_t launch_tile_kernel(int kind, const CUtensorMap& map_a, const CUtensorMap& map_b,
                               const TileParams& p, int num_sms, cudaStream_t stream) {
    if (p.n_items <= 0) return cudaSuccess;
    const int smem = (int)sizeof(Shared) + 1024;
    const int grid = p.n_items < num_sms ? p.n_items : num_sms;
    cudaError_t err;
#define LOOKM_LAUNCH(K)                                                                          \
    err = cudaFuncSetAttribute(tile_kernel<K>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem); \
    if (err != cudaSuccess) return err;                                                          \
    tile_kernel<K><<<grid, kThreads, smem, stream>>>(map_a, map_b, p);
    if (kind == kSweep1) { LOOKM_LAUNCH(kSweep1) }
    else if (kind == kSweep2) { LOOKM_LAUNCH(kSweep2) }
    else { LOOKM_LAUNCH(kMatch) }
#undef LOOKM_LAUNCH
    return cudaGetLastError();
}

}  // namespace lookm
