// Bandwidth-bound kernels of the path: key norms, compaction of the kept keys (the B operand of
// the matching), row arg-max of given similarity matrices, inversion of the evicted->kept
// assignment into per-kept-row member lists, and the merge/compact kernel (Eq. 6-7, 10-12).
//
// A K or V row is 128 bf16 = 256 bytes = 16 lanes x 16 bytes, so a half-warp moves one row with
// one 16-byte access per lane.
#include <cuda_bf16.h>

#include "internal.h"

namespace lookm {
namespace {

struct Row8 { float v[8]; };

__device__ __forceinline__ Row8 unpack8(const uint4& u) {
    Row8 r;
    const unsigned w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        r.v[2 * i] = __uint_as_float(w[i] << 16);
        r.v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    return r;
}

__device__ __forceinline__ uint4 pack8(const Row8& r) {
    unsigned w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 b = __floats2bfloat162_rn(r.v[2 * i], r.v[2 * i + 1]);
        w[i] = *reinterpret_cast<const unsigned*>(&b);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ const Req& find_req_by_slot(const Req* reqs, int n_req, long long g) {
    int lo = 0, hi = n_req - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if ((long long)reqs[mid].slot_begin <= g) lo = mid; else hi = mid - 1;
    }
    return reqs[lo];
}

// ---------------------------------------------------------------------------------------------
// 1 / |k| of every key row (0 for a zero row), the cosine denominators of Eq. 9.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
key_norms_kernel(const __nv_bfloat16* __restrict__ k, long long stride_tok, long long stride_head,
                 int n_kv_heads, long long T, float* __restrict__ rnorm_all) {
    const int half = threadIdx.x >> 4, l16 = threadIdx.x & 15;
    const long long n_rows = T * n_kv_heads;
    // the loop bound is the warp's first row, so that both half-warps always reach the shuffles
    for (long long rw = (long long)blockIdx.x * 16 + (half & ~1); rw < n_rows; rw += (long long)gridDim.x * 16) {
        const long long r = rw + (half & 1);
        const bool valid = r < n_rows;
        const long long tok = valid ? r / n_kv_heads : 0;
        const int h = valid ? (int)(r % n_kv_heads) : 0;
        const uint4 u = *reinterpret_cast<const uint4*>(k + tok * stride_tok + h * stride_head + l16 * 8);
        const Row8 x = unpack8(u);
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) ss = fmaf(x.v[i], x.v[i], ss);
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o, 16);
        if (l16 == 0 && valid) rnorm_all[(long long)h * T + tok] = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
    }
}

// ---------------------------------------------------------------------------------------------
// Kept keys of every (request, head) copied into one dense [rows, 128] matrix in kept-list
// order, with their inverse norms.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
gather_kept_kernel(const __nv_bfloat16* __restrict__ k, long long stride_tok, long long stride_head,
                   const Req* __restrict__ reqs, int n_req, int n_kv_heads, long long T,
                   long long total_rows, const int* __restrict__ kept_idx,
                   const float* __restrict__ rnorm_all, __nv_bfloat16* __restrict__ kept_keys,
                   float* __restrict__ rnorm_kept, int* status) {
    grid_dependency_wait();
    const int half = threadIdx.x >> 4, l16 = threadIdx.x & 15;
    const long long g = (long long)blockIdx.x * 16 + half;
    if (g >= total_rows) return;
    const Req& rq = find_req_by_slot(reqs, n_req, g);
    if (rq.mode == LOOKM_MERGE_NONE) return;             // nothing is matched against its kept keys
    const long long u = g - rq.slot_begin;
    const int h = (int)(u / rq.B), slot = (int)(u % rq.B);
    const long long dst = rq.kept_off + (long long)h * rq.B + slot;
    int pos = kept_idx[dst];
    if (pos < 0 || pos >= rq.L) { if (l16 == 0) atomicExch(status, (int)LOOKM_ERR_DEVICE_BAD_INDEX); pos = 0; }
    const long long tok = rq.tok_begin + pos;
    const uint4 u4 = *reinterpret_cast<const uint4*>(k + tok * stride_tok + h * stride_head + l16 * 8);
    *reinterpret_cast<uint4*>(kept_keys + dst * kHeadDim + l16 * 8) = u4;
    if (l16 == 0) rnorm_kept[dst] = rnorm_all[(long long)h * T + tok];
}

// ---------------------------------------------------------------------------------------------
// Eviction alone (Eq. 6-7): kept K and V rows of the requests with LOOKM_MERGE_NONE copied to the
// output cache, one warp per row (lanes 0-15 the K row, 16-31 the V row).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
compact_kept_kernel(const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                    long long stride_tok, long long stride_head, const Req* __restrict__ reqs, int n_req,
                    int n_kv_heads, long long total_rows, const int* __restrict__ kept_idx,
                    int varlen_output, long long out_stride_head, __nv_bfloat16* __restrict__ out_k,
                    __nv_bfloat16* __restrict__ out_v, int* status) {
    grid_dependency_wait();
    const int lane = threadIdx.x & 31, l16 = lane & 15;
    const long long g = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (g >= total_rows) return;
    const Req& rq = find_req_by_slot(reqs, n_req, g);
    if (rq.mode != LOOKM_MERGE_NONE) return;
    const long long u = g - rq.slot_begin;
    const int h = (int)(u / rq.B), slot = (int)(u % rq.B);
    int pos = kept_idx[rq.kept_off + (long long)h * rq.B + slot];
    if (pos < 0 || pos >= rq.L) { if (lane == 0) atomicExch(status, (int)LOOKM_ERR_DEVICE_BAD_INDEX); pos = 0; }
    const __nv_bfloat16* src = (lane < 16 ? k : v) + (rq.tok_begin + (long long)pos) * stride_tok +
                               (long long)h * stride_head + l16 * 8;
    long long dst;
    if (varlen_output) dst = (((long long)rq.out_begin + slot) * n_kv_heads + h) * kHeadDim;
    else dst = (long long)h * out_stride_head + (long long)slot * kHeadDim;
    *reinterpret_cast<uint4*>((lane < 16 ? out_k : out_v) + dst + l16 * 8) = *reinterpret_cast<const uint4*>(src);
}

// ---------------------------------------------------------------------------------------------
// Row arg-max of given similarity blocks (one warp per evicted row); lowest slot wins ties.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
argmax_rows_kernel(const float* __restrict__ sim_matrix, const Req* __restrict__ reqs,
                   int n_kv_heads, int* __restrict__ assign, float* __restrict__ sim) {
    const Req rq = reqs[blockIdx.z];
    const int h = blockIdx.y;
    const int e = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (e >= rq.E) return;
    const float* row = sim_matrix + rq.sim_off + ((long long)h * rq.E + e) * rq.B;
    float best = -INFINITY;
    int slot = 0x7fffffff;
    for (int c = lane; c < rq.B; c += 32) {
        const float v = row[c];
        if (v > best) { best = v; slot = c; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int os = __shfl_xor_sync(0xffffffffu, slot, o);
        if (ob > best || (ob == best && os < slot)) { best = ob; slot = os; }
    }
    if (lane == 0) {
        assign[rq.ev_off + (long long)h * rq.E + e] = slot;
        sim[rq.ev_off + (long long)h * rq.E + e] = best;
    }
}

// ---------------------------------------------------------------------------------------------
// Inversion of the assignment: for each (request, head) a stable sort of the evicted ranks by
// their kept slot gives, per kept row, its members in ascending position, as CSR
// (row_ptr [B + 1 per (request, head)], member positions and weights [E]).  One CTA per (request, head); stable LSD
// radix sort with 8-bit digits: every warp owns a contiguous segment of the list, ranks equal
// digits inside a 32-element step with match.any, and adds the counts of earlier steps and
// earlier warps.  Keys are packed as (slot << 0) in one array and values in the other.
// ---------------------------------------------------------------------------------------------
constexpr int kInvThreads = 1024;

// Second half of the entry list: the kept rows (flagged with the sign bit, weight = member count),
// for every work unit (unit u of a head covers the entries [u * unit_entries, (u + 1) * unit_entries))
// the slot its first entry belongs to, with that slot's first entry and member count, and a
// cleared arrival counter per slot.
__device__ __forceinline__ void write_kept_entries(const Req& rq, int h, int n_kv_heads, int B, const int* rp,
                                                   const int* kept_idx_head, int* ent, float* entw,
                                                   int4* unit_first, int* slot_cnt, int* status) {
    const int ue = rq.unit_entries;
    for (int c = threadIdx.x; c < B; c += blockDim.x) {
        int pc = kept_idx_head[c];
        if (pc < 0 || pc >= rq.L) { atomicExch(status, (int)LOOKM_ERR_DEVICE_BAD_INDEX); pc = 0; }
        const int s_c = c + rp[c];                       // entry of the kept row
        const int s_next = c + 1 + rp[c + 1];            // entry of the next kept row (L after the last)
        ent[s_c] = pc | (int)0x80000000;
        entw[s_c] = (float)(rp[c + 1] - rp[c]);
        slot_cnt[c] = 0;
        for (int u = (s_c + ue - 1) / ue; u * ue < s_next; ++u)
            unit_first[(long long)u * n_kv_heads + h] = make_int4(c, s_c, rp[c + 1] - rp[c], 0);
    }
}

// Lanes of the warp that hold a valid element with the same digit as the caller: one ballot per
// digit bit (match.any takes a step per distinct value, i.e. up to 32 for well-mixed digits).
__device__ __forceinline__ unsigned same_digit_lanes(unsigned d, bool valid, int dbits) {
    unsigned peers = __ballot_sync(0xffffffffu, valid);
#pragma unroll
    for (int b = 0; b < kInvDigitBits16; ++b) {
        if (b < dbits) {
            const bool bit = (d >> b) & 1u;
            const unsigned bal = __ballot_sync(0xffffffffu, bit);
            peers &= bit ? bal : ~bal;
        }
    }
    return peers;
}

constexpr int kInvBatch = 8;                         // loop steps whose loads are issued together

// CountT / kMaxBits: 16-bit counters with digits of up to 11 bits when no request of the call evicts
// more than 65535 tokens per head (every count and prefix then fits), else 32-bit counters with
// digits of up to 10 bits; either way at most 136 KB of counters per CTA.
template <typename CountT, int kMaxBits>
__global__ void __launch_bounds__(kInvThreads)
invert_assignment_kernel(const int* __restrict__ assign, const int* __restrict__ kept_idx,
                         const int* __restrict__ evict_idx,
                         const float* __restrict__ sim, const Req* __restrict__ reqs,
                         int n_kv_heads, long long T, int* __restrict__ row_ptr,
                         int* __restrict__ ent_pos, float* __restrict__ ent_w,
                         int4* __restrict__ unit_first, int* __restrict__ slot_cnt,
                         unsigned* __restrict__ sort_a, unsigned* __restrict__ sort_b, int* status) {
    extern __shared__ __align__(16) unsigned char inv_smem[];
    __shared__ int warp_sums[32];
    grid_dependency_wait();
    const Req rq = reqs[blockIdx.y];
    if (rq.mode == LOOKM_MERGE_NONE) return;             // its kept rows are copied, nothing is merged
    const int h = blockIdx.x;
    const int E = rq.E, B = rq.B;
    const long long ev_base = rq.ev_off + (long long)h * E;
    int* rp = row_ptr + rq.rp_off + (long long)h * (B + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned lt_mask = (1u << lane) - 1u;

    // entry list of this (request, head): for every kept slot its kept row, then its members
    int* ent = ent_pos + (long long)h * T + rq.tok_begin;
    float* entw = ent_w + (long long)h * T + rq.tok_begin;
    int4* units = unit_first + rq.unit_begin;            // [unit of the head][head]
    int* cnts = slot_cnt + rq.kept_off + (long long)h * B;
    const int* kept_idx_head = kept_idx + rq.kept_off + (long long)h * B;
    const bool weighted = (rq.mode == LOOKM_MERGE_WEIGHTED);
    if (E == 0) {
        for (int c = threadIdx.x; c <= B; c += kInvThreads) rp[c] = 0;
        __syncthreads();
        write_kept_entries(rq, h, n_kv_heads, B, rp, kept_idx_head, ent, entw, units, cnts, status);
        return;
    }
    // segment of the list owned by each warp: a multiple of 32 elements
    const int seg = ((E + 32 * 32 - 1) / (32 * 32)) * 32;
    const int s_begin = min(E, warp * seg), s_end = min(E, s_begin + seg);

    int n_pass, dbits;
    invert_digits(B, kMaxBits, n_pass, dbits);
    const int nd = 1 << dbits;
    const unsigned dmask = (unsigned)nd - 1u;
    CountT* cnt = reinterpret_cast<CountT*>(inv_smem);                          // [warp][digit]
    int* digit_tot = reinterpret_cast<int*>(inv_smem + (size_t)32 * nd * sizeof(CountT));
    const bool single = (n_pass == 1);
    // One pass over a segment of at most kInvBatch steps per warp: the count phase already knows
    // every element's rank among the equal slots of its warp, so the scatter phase needs neither
    // the ballots nor the running counts again.
    const bool keep_ranks = single && seg <= 32 * kInvBatch;
    int local_rank[kInvBatch];
#pragma unroll
    for (int q = 0; q < kInvBatch; ++q) local_rank[q] = 0;

    // pass p reads (key, value) from src and writes to dst; pass 0 reads assign directly.  With a
    // single pass the sorted position is final, and the entries are written straight away.
    unsigned* key_buf[2] = {sort_a + 2 * ev_base, sort_b + 2 * ev_base};   // [E keys][E values] each
    for (int pass = 0; pass < n_pass; ++pass) {
        const int shift = pass * dbits;
        const unsigned* src_k = pass ? key_buf[(pass - 1) & 1] : nullptr;
        const unsigned* src_v = pass ? key_buf[(pass - 1) & 1] + E : nullptr;
        unsigned* dst_k = key_buf[pass & 1];
        unsigned* dst_v = key_buf[pass & 1] + E;
        for (int i = threadIdx.x; i < (int)(32 * sizeof(CountT) / 4) * nd; i += kInvThreads)
            reinterpret_cast<unsigned*>(cnt)[i] = 0u;
        __syncthreads();
        // count (the loads of kInvBatch steps are issued together: the loop is bound by their latency)
        for (int b0 = s_begin; b0 < s_end; b0 += 32 * kInvBatch) {
            unsigned key[kInvBatch];
#pragma unroll
            for (int q = 0; q < kInvBatch; ++q) {
                const int i = b0 + q * 32 + lane;
                key[q] = 0u;
                if (i < s_end) key[q] = pass ? src_k[i] : (unsigned)assign[ev_base + i];
            }
#pragma unroll
            for (int q = 0; q < kInvBatch; ++q) {
                const int i = b0 + q * 32 + lane;
                const bool valid = i < s_end;
                if (valid && !pass && key[q] >= (unsigned)B) {
                    atomicExch(status, (int)LOOKM_ERR_DEVICE_BAD_INDEX);
                    key[q] = 0u;
                }
                const unsigned d = (key[q] >> shift) & dmask;
                const unsigned peers = same_digit_lanes(d, valid, dbits);
                if (keep_ranks) {
                    local_rank[q] = valid ? (int)cnt[warp * nd + d] + __popc(peers & lt_mask) : 0;
                    __syncwarp();
                }
                if (valid && (peers & lt_mask) == 0u) cnt[warp * nd + d] += (CountT)__popc(peers);
                __syncwarp();
            }
        }
        __syncthreads();
        // exclusive scan over (digit major, warp minor): first over the warps of every digit ...
        for (int d = threadIdx.x; d < nd; d += kInvThreads) {
            int tot = 0;
            for (int w = 0; w < 32; ++w) {
                const int c = cnt[w * nd + d];
                cnt[w * nd + d] = (CountT)tot;
                tot += c;
            }
            digit_tot[d] = tot;
        }
        __syncthreads();
        // ... then over the digit totals (two digits per thread; nd <= 2 * kInvThreads)
        {
            const int d0 = 2 * threadIdx.x;
            const int a = d0 < nd ? digit_tot[d0] : 0;
            const int b = d0 + 1 < nd ? digit_tot[d0 + 1] : 0;
            int incl = a + b;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int x = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += x;
            }
            if (lane == 31) warp_sums[warp] = incl;
            __syncthreads();
            if (warp == 0) {
                int ws = warp_sums[lane];
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int x = __shfl_up_sync(0xffffffffu, ws, o);
                    if (lane >= o) ws += x;
                }
                warp_sums[lane] = ws;
            }
            __syncthreads();
            const int base = (warp ? warp_sums[warp - 1] : 0) + incl - (a + b);
            if (d0 < nd) digit_tot[d0] = base;
            if (d0 + 1 < nd) digit_tot[d0 + 1] = base + a;
        }
        __syncthreads();
        if (single) {
            // row boundaries: row_ptr[c] = first sorted index whose slot is >= c
            for (int c = threadIdx.x; c <= B; c += kInvThreads) rp[c] = c < nd ? digit_tot[c] : E;
        }
        // scatter
        for (int b0 = s_begin; b0 < s_end; b0 += 32 * kInvBatch) {
            unsigned key[kInvBatch], val[kInvBatch];
            int pe[kInvBatch];
            float w[kInvBatch];
#pragma unroll
            for (int q = 0; q < kInvBatch; ++q) {
                const int i = b0 + q * 32 + lane;
                key[q] = 0u;
                val[q] = (unsigned)i;
                pe[q] = 0;
                w[q] = 1.0f;
                if (i < s_end) {
                    if (pass) { key[q] = src_k[i]; val[q] = src_v[i]; }
                    else key[q] = (unsigned)assign[ev_base + i];
                    if (single) {
                        pe[q] = evict_idx[ev_base + i];
                        if (weighted) w[q] = sim[ev_base + i];
                    }
                }
            }
#pragma unroll
            for (int q = 0; q < kInvBatch; ++q) {
                const int i = b0 + q * 32 + lane;
                const bool valid = i < s_end;
                if (!pass && key[q] >= (unsigned)B) key[q] = 0u;
                const unsigned d = (key[q] >> shift) & dmask;
                int off = 0;
                if (keep_ranks) {
                    if (valid) off = digit_tot[d] + (int)cnt[warp * nd + d] + local_rank[q];
                } else {
                    const unsigned peers = same_digit_lanes(d, valid, dbits);
                    if (valid) off = digit_tot[d] + (int)cnt[warp * nd + d] + __popc(peers & lt_mask);
                    __syncwarp();
                    if (valid && (peers & lt_mask) == 0u) cnt[warp * nd + d] += (CountT)__popc(peers);
                    __syncwarp();
                }
                if (valid) {
                    if (single) {
                        if (pe[q] < 0 || pe[q] >= rq.L) { atomicExch(status, (int)LOOKM_ERR_DEVICE_BAD_INDEX); pe[q] = 0; }
                        ent[off + (int)key[q] + 1] = pe[q];      // sits after key + 1 kept rows
                        entw[off + (int)key[q] + 1] = w[q];
                    } else {
                        dst_k[off] = key[q];
                        dst_v[off] = val[q];
                    }
                }
            }
        }
        __syncthreads();
    }
    if (!single) {
        const unsigned* fin_k = key_buf[(n_pass - 1) & 1];
        const unsigned* fin_v = fin_k + E;
        // member entries and the row boundaries: row_ptr[c] = first sorted index whose slot is >= c
        for (int i0 = threadIdx.x; i0 < E; i0 += kInvThreads * kInvBatch) {
            int e[kInvBatch], cur[kInvBatch], prev[kInvBatch], pe[kInvBatch];
            float w[kInvBatch];
#pragma unroll
            for (int q = 0; q < kInvBatch; ++q) {
                const int i = i0 + q * kInvThreads;
                e[q] = 0; cur[q] = 0; prev[q] = -1;
                if (i < E) {
                    e[q] = (int)fin_v[i];
                    cur[q] = (int)fin_k[i];
                    if (i) prev[q] = (int)fin_k[i - 1];
                }
            }
#pragma unroll
            for (int q = 0; q < kInvBatch; ++q) {
                const int i = i0 + q * kInvThreads;
                pe[q] = 0; w[q] = 1.0f;
                if (i < E) {
                    pe[q] = evict_idx[ev_base + e[q]];
                    if (weighted) w[q] = sim[ev_base + e[q]];
                }
            }
#pragma unroll
            for (int q = 0; q < kInvBatch; ++q) {
                const int i = i0 + q * kInvThreads;
                if (i >= E) continue;
                if (pe[q] < 0 || pe[q] >= rq.L) { atomicExch(status, (int)LOOKM_ERR_DEVICE_BAD_INDEX); pe[q] = 0; }
                ent[i + cur[q] + 1] = pe[q];             // i-th member sits after cur + 1 kept rows
                entw[i + cur[q] + 1] = w[q];
                for (int c = prev[q] + 1; c <= cur[q]; ++c) rp[c] = i;
                if (i == E - 1) for (int c = cur[q] + 1; c <= B; ++c) rp[c] = E;
            }
        }
    }
    __syncthreads();
    write_kept_entries(rq, h, n_kv_heads, B, rp, kept_idx_head, ent, entw, units, cnts, status);
}

// ---------------------------------------------------------------------------------------------
// Merge + compact (Eq. 6-7, 10-12).  Every K and V row of the prompt is read exactly once: the
// entry list of a (request, head) names, slot by slot, the kept row and then its members.  A warp
// takes a work unit of unit_entries consecutive entries (sized so that each warp gets about one
// unit, at least 32 entries), fetches the rows 8 entries at a time with 16-byte cp.async copies
// into its own shared-memory ring (three buffers; every lane later reads back exactly the bytes it
// copied, so cp.async.wait_group is all the synchronisation needed), and walks the staged rows in
// order: lanes 0-15 hold the K row, lanes 16-31 the V row, 16 bytes per lane, fp32 accumulation in
// member order, one rounding.
//   averaged : (x_c + sum x_e) / (n + 1)                       (Eq. 10)
//   pivotal  : (x_c + 1/2 sum (x_e + x_c)) / (n + 1)           (Eq. 11)
//   weighted : (x_c + sum sim_e x_e) / (n + 1)                 (Eq. 12)
// A row without members is copied bit for bit.
//
// Units are cut at fixed entry counts, not at slot boundaries, so that every warp has the same
// amount to read however skewed the member counts are.  A slot whose entries straddle units is
// summed piecewise: every unit that holds a piece stores its fp32 partial sum (the unit with the
// kept row also stores that row) in its own record, then bumps the slot's arrival counter; the
// warp that arrives last adds the pieces in unit order and writes the row.  Nobody waits for
// anybody, and the order of the additions does not depend on who came last.
// ---------------------------------------------------------------------------------------------
constexpr int kMergeWarps = 16;                      // per CTA; one CTA per SM
constexpr int kChunk = 8;                            // entries staged per buffer
constexpr int kRing = 3;                             // buffers per warp: two chunks in flight while one is read
constexpr int kRowBytes = kHeadDim * 2;              // one bf16 row of K or V
// Record of a unit: [0, 1024) partial sums of its leading piece (slot begun in an earlier unit),
// [1024, 2048) partial sums of its trailing piece (slot that goes on in the next unit),
// [2048, 2560) the kept K|V row of the trailing piece.  Per piece: 8 floats (or 16 bytes) per lane.
constexpr int kPartFloats = kMergePartBytes / 4;

struct MergeShared {
    alignas(128) uint8_t rows[kMergeWarps][kRing][kChunk][2 * kRowBytes];   // [warp][buffer][entry][K|V]
};

__device__ __forceinline__ const Req& find_req_by_unit(const Req* reqs, int n_req, long long g) {
    int lo = 0, hi = n_req - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if ((long long)reqs[mid].unit_begin <= g) lo = mid; else hi = mid - 1;
    }
    return reqs[lo];
}

__device__ __forceinline__ float4 ld_cg_f4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

__global__ void __launch_bounds__(kMergeWarps * 32)
merge_kernel(const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
             long long stride_tok, long long stride_head, const Req* __restrict__ reqs, int n_req,
             int n_kv_heads, long long T, long long total_units, const int* __restrict__ row_ptr,
             const int* __restrict__ ent_pos, const float* __restrict__ ent_w,
             const int4* __restrict__ unit_first, int* __restrict__ slot_cnt, float* __restrict__ parts,
             int varlen_output, long long out_stride_head, __nv_bfloat16* __restrict__ out_k,
             __nv_bfloat16* __restrict__ out_v, int* status) {
    extern __shared__ uint8_t merge_smem_raw[];
    MergeShared& sh = *reinterpret_cast<MergeShared*>(
        (reinterpret_cast<uintptr_t>(merge_smem_raw) + 127) & ~static_cast<uintptr_t>(127));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int l16 = lane & 15;
    const uint32_t buf0 = (uint32_t)__cvta_generic_to_shared(&sh.rows[warp][0][0][0]) + lane * 16;
    const __nv_bfloat16* tensor = lane < 16 ? k : v;
    __nv_bfloat16* dst_base = lane < 16 ? out_k : out_v;
    const unsigned tok_bytes = (unsigned)stride_tok * 2u;      // the launcher checks that this fits
    uint32_t n_chunks_done = 0;                      // chunks this warp has consumed (buffer parity)
    grid_dependency_wait();

    for (long long g = (long long)blockIdx.x * kMergeWarps + warp; g < total_units;
         g += (long long)gridDim.x * kMergeWarps) {
        const Req& rq = find_req_by_unit(reqs, n_req, g);
        const int L = rq.L, B = rq.B, mode = rq.mode, ue = rq.unit_entries;
        const long long ul = g - rq.unit_begin;
        // heads vary fastest: warps running at the same time then read the same token range of
        // different heads, i.e. neighbouring 256-byte rows of the same DRAM pages
        const int h = (int)(ul % n_kv_heads), u = (int)(ul / n_kv_heads);
        const int e_lo = u * ue, e_hi = min(L, e_lo + ue);
        int4 first = make_int4(0, 0, 0, 0);           // slot of the first entry; its first entry, member count
        if (lane == 0) first = __ldg(unit_first + g); // needed at the first kept row at the earliest
        int* cnt = slot_cnt + rq.kept_off + (long long)h * B;
        const int* ent = ent_pos + (long long)h * T + rq.tok_begin;
        const float* entw = ent_w + (long long)h * T + rq.tok_begin;
        const char* src = reinterpret_cast<const char*>(tensor + (long long)rq.tok_begin * stride_tok +
                                                        (long long)h * stride_head + l16 * 8);
        const int n_chunks = (e_hi - e_lo + kChunk - 1) / kChunk;

        // entry metadata of a chunk (lanes 0-7: one entry each)
        auto load_meta = [&](int kc, int& pos, float& w) {
            pos = 0;
            w = 0.f;
            const int e = e_lo + kc * kChunk + lane;
            if (lane < kChunk && kc < n_chunks && e < e_hi) { pos = ent[e]; w = entw[e]; }
        };
        // start the row copies of chunk kc: for every entry, lanes 0-15 copy its K row and lanes
        // 16-31 its V row, 16 bytes each; one commit group per chunk
        auto issue = [&](int kc, int pos) {
            const int n_ent = min(kChunk, e_hi - e_lo - kc * kChunk);    // <= 0 past the unit: empty group
            const uint32_t dst = buf0 + ((n_chunks_done + (uint32_t)kc) % kRing) * (kChunk * 2 * kRowBytes);
#pragma unroll
            for (int q = 0; q < kChunk; ++q) {
                const unsigned tok = (unsigned)__shfl_sync(0xffffffffu, pos, q) & 0x7fffffffu;
                if (q < n_ent)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                                 ::"r"(dst + q * (2 * kRowBytes)), "l"(src + (size_t)tok * tok_bytes)
                                 : "memory");
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };

        int pos_a, pos_b, pos_c;
        float w_a, w_b, w_c;
        load_meta(0, pos_a, w_a);
        load_meta(1, pos_b, w_b);
        load_meta(2, pos_c, w_c);
        issue(0, pos_a);
        issue(1, pos_b);

        // running piece: the slot, whether its kept row was met in this unit (and at which entry),
        // the members met
        const bool starts_with_kept = __shfl_sync(0xffffffffu, pos_a, 0) < 0;
        const int first_slot = __shfl_sync(0xffffffffu, first.x, 0);
        int slot = starts_with_kept ? first_slot - 1 : first_slot;
        bool active = !starts_with_kept, have_kept = false;
        bool lead_piece = false, trail_piece = false;    // pieces of shared slots this unit has stored
        int n_mem = 0, n_seen = 0, kept_entry = 0;
        uint4 raw_c = make_uint4(0u, 0u, 0u, 0u);
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;

        auto write_row = [&](int c, const uint4& kept_raw, const float* sum, int n) {
            uint4 result = kept_raw;
            if (n > 0) {
                const Row8 xc = unpack8(kept_raw);
                const float inv = 1.0f / (float)(n + 1);
                // pivotal: each member contributes (x_e + x_c) / 2
                const float wc = (mode == LOOKM_MERGE_PIVOTAL) ? 1.f + 0.5f * (float)n : 1.f;
                const float wm = (mode == LOOKM_MERGE_PIVOTAL) ? 0.5f : 1.f;
                Row8 o;
#pragma unroll
                for (int i = 0; i < 8; ++i) o.v[i] = fmaf(wc, xc.v[i], wm * sum[i]) * inv;
                result = pack8(o);
            }
            long long at;
            if (varlen_output) at = (((long long)rq.out_begin + c) * n_kv_heads + h) * kHeadDim;
            else at = (long long)h * out_stride_head + (long long)c * kHeadDim;
            *reinterpret_cast<uint4*>(dst_base + at + l16 * 8) = result;
        };
        // ends the running piece: a whole slot is written out; a piece of a slot that other units
        // share goes to this unit's record (announced after the loop)
        auto flush = [&]() {
            if (!active) return;
            if (have_kept && n_seen == n_mem) {
                write_row(slot, raw_c, acc, n_mem);
                return;
            }
            float* rec = parts + g * kPartFloats + (have_kept ? 256 : 0) + lane * 8;
            *reinterpret_cast<float4*>(rec) = make_float4(acc[0], acc[1], acc[2], acc[3]);
            *reinterpret_cast<float4*>(rec + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
            if (have_kept) {
                *reinterpret_cast<uint4*>(parts + g * kPartFloats + 512 + lane * 4) = raw_c;
                trail_piece = true;
            } else {
                lead_piece = true;
            }
        };
        // adds the pieces of slot c (kept row in unit u0, last member in unit u1) in unit order
        auto combine = [&](int c, int u0, int u1, int n) {
            const float* r0 = parts + ((long long)rq.unit_begin + (long long)u0 * n_kv_heads + h) * kPartFloats;
            float sum[8];
            {
                const float4 lo = ld_cg_f4(r0 + 256 + lane * 8), hi = ld_cg_f4(r0 + 256 + lane * 8 + 4);
                sum[0] = lo.x; sum[1] = lo.y; sum[2] = lo.z; sum[3] = lo.w;
                sum[4] = hi.x; sum[5] = hi.y; sum[6] = hi.z; sum[7] = hi.w;
            }
            const uint4 kept_raw = __ldcg(reinterpret_cast<const uint4*>(r0 + 512 + lane * 4));
            for (int uu = u0 + 1; uu <= u1; ++uu) {
                const float* r = r0 + (long long)(uu - u0) * n_kv_heads * kPartFloats;
                const float4 lo = ld_cg_f4(r + lane * 8), hi = ld_cg_f4(r + lane * 8 + 4);
                sum[0] += lo.x; sum[1] += lo.y; sum[2] += lo.z; sum[3] += lo.w;
                sum[4] += hi.x; sum[5] += hi.y; sum[6] += hi.z; sum[7] += hi.w;
            }
            write_row(c, kept_raw, sum, n);
        };

        for (int kc = 0; kc < n_chunks; ++kc) {
            // chunk kc + 2 goes to the buffer whose rows were consumed one iteration ago; a commit
            // group is made for every chunk index (empty past the unit), so "all but the two
            // newest groups" always means: chunk kc has landed
            issue(kc + 2, pos_c);
            int pos_d;
            float w_d;
            load_meta(kc + 3, pos_d, w_d);
            asm volatile("cp.async.wait_group 2;" ::: "memory");
            const int n_ent = min(kChunk, e_hi - e_lo - kc * kChunk);
            const uint32_t rows = buf0 + ((n_chunks_done + (uint32_t)kc) % kRing) * (kChunk * 2 * kRowBytes);
            uint4 x[kChunk];                         // this lane's 16 bytes of every staged row
#pragma unroll
            for (int q = 0; q < kChunk; ++q)
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(x[q].x), "=r"(x[q].y), "=r"(x[q].z), "=r"(x[q].w)
                             : "r"(rows + q * (2 * kRowBytes)));
#pragma unroll
            for (int q = 0; q < kChunk; ++q) {
                const int pe = __shfl_sync(0xffffffffu, pos_a, q);
                const float w = __shfl_sync(0xffffffffu, w_a, q);
                if (q >= n_ent) break;
                if (pe < 0) {                        // a kept row starts the next slot
                    flush();
                    ++slot;
                    active = true;
                    have_kept = true;
                    raw_c = x[q];
                    n_mem = (int)w;
                    n_seen = 0;
                    kept_entry = e_lo + kc * kChunk + q;
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
                } else {
                    const Row8 xe = unpack8(x[q]);
                    ++n_seen;
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[i] = fmaf(w, xe.v[i], acc[i]);
                }
            }
            __syncwarp();
            pos_a = pos_b; w_a = w_b;
            pos_b = pos_c; w_b = w_c;
            pos_c = pos_d; w_c = w_d;
        }
        flush();
        n_chunks_done += (uint32_t)n_chunks;
        if (lead_piece || trail_piece) {
            // announce the stored pieces (lane 0: the leading one, lane 1: the trailing one); the
            // unit that arrives last at a slot finishes its row
            __threadfence();
            __syncwarp();
            int c = 0, s0 = 0, n = 0;
            bool mine = false;
            if (lane == 0 && lead_piece) { c = first.x; s0 = first.y; n = first.z; mine = true; }
            if (lane == 1 && trail_piece) { c = slot; s0 = kept_entry; n = n_mem; mine = true; }
            const int u0 = s0 / ue, u1 = (s0 + n) / ue;          // units of the kept row / the last member
            const bool last = mine && atomicAdd(cnt + c, 1) == u1 - u0;
            const unsigned finish = __ballot_sync(0xffffffffu, last);
            if (finish) __threadfence();
            for (int which = 0; which < 2; ++which)
                if (finish & (1u << which))
                    combine(__shfl_sync(0xffffffffu, c, which), __shfl_sync(0xffffffffu, u0, which),
                            __shfl_sync(0xffffffffu, u1, which), __shfl_sync(0xffffffffu, n, which));
        }
    }
    (void)status;
}

__global__ void write_table_kernel(const __grid_constant__ ReqChunk chunk, int count, Req* dst) {
    const int i = threadIdx.x;
    if (i < count) dst[i] = chunk.r[i];
}

}  // namespace

cudaError_t launch_write_table(const ReqChunk& chunk, int count, Req* dst, cudaStream_t stream) {
    write_table_kernel<<<1, 64, 0, stream>>>(chunk, count, dst);
    return cudaGetLastError();
}

cudaError_t launch_key_norms(const void* k, long long stride_tok, long long stride_head,
                             int n_kv_heads, long long T, float* rnorm_all, cudaStream_t stream) {
    const long long rows = T * n_kv_heads;
    if (rows <= 0) return cudaSuccess;
    long long blocks = (rows + 15) / 16;
    if (blocks > 148 * 32) blocks = 148 * 32;
    key_norms_kernel<<<(int)blocks, 256, 0, stream>>>((const __nv_bfloat16*)k, stride_tok, stride_head,
                                                      n_kv_heads, T, rnorm_all);
    return cudaGetLastError();
}

cudaError_t launch_gather_kept(const void* k, long long stride_tok, long long stride_head,
                               const Req* reqs, int n_req, int n_kv_heads, long long T,
                               long long total_kept_rows, const int* kept_idx,
                               const float* rnorm_all, void* kept_keys, float* rnorm_kept,
                               int* status, cudaStream_t stream) {
    if (total_kept_rows <= 0) return cudaSuccess;
    const long long blocks = (total_kept_rows + 15) / 16;
    return launch_chained(gather_kept_kernel, dim3((unsigned)blocks), dim3(256), 0, stream,
                          (const __nv_bfloat16*)k, stride_tok, stride_head, reqs, n_req, n_kv_heads, T,
                          total_kept_rows, kept_idx, rnorm_all, (__nv_bfloat16*)kept_keys, rnorm_kept,
                          status);
}

cudaError_t launch_invert_assignment(const int* assign, const int* kept_idx, const int* evict_idx,
                                     const float* sim, const Req* reqs, int n_req, int n_kv_heads,
                                     long long T, bool wide_counts, int digit_bits, int* row_ptr,
                                     int* ent_pos, float* ent_w, int4* unit_first, int* slot_cnt,
                                     unsigned* sort_a, unsigned* sort_b, int* status,
                                     cudaStream_t stream) {
    // counters of the widest digit any request of the call needs: 32 warps x 2^digit_bits counts
    // and 2^digit_bits totals
    const size_t smem = ((size_t)32 * (wide_counts ? sizeof(unsigned) : sizeof(unsigned short)) + sizeof(int))
                        << digit_bits;
    dim3 grid(n_kv_heads, n_req);
    // the shared-memory limit is raised once per device to the most either instantiation can ask
    // for (32 warps x 2^bits counters and 2^bits totals)
    static unsigned long long configured = 0;
    cudaError_t err = once_per_device(configured, [&]() {
        const int max16 = (int)(((size_t)32 * sizeof(unsigned short) + sizeof(int)) << kInvDigitBits16);
        const int max32 = (int)(((size_t)32 * sizeof(unsigned) + sizeof(int)) << kInvDigitBits32);
        cudaError_t e = cudaFuncSetAttribute(invert_assignment_kernel<unsigned short, kInvDigitBits16>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, max16);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(invert_assignment_kernel<unsigned, kInvDigitBits32>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, max32);
        return e;
    });
    if (err != cudaSuccess) return err;
    if (wide_counts)
        return launch_chained(invert_assignment_kernel<unsigned, kInvDigitBits32>, grid, dim3(kInvThreads), smem,
                              stream, assign, kept_idx, evict_idx, sim, reqs, n_kv_heads, T, row_ptr, ent_pos,
                              ent_w, unit_first, slot_cnt, sort_a, sort_b, status);
    return launch_chained(invert_assignment_kernel<unsigned short, kInvDigitBits16>, grid, dim3(kInvThreads), smem,
                          stream, assign, kept_idx, evict_idx, sim, reqs, n_kv_heads, T, row_ptr, ent_pos,
                          ent_w, unit_first, slot_cnt, sort_a, sort_b, status);
}

int merge_warps_per_sm() { return kMergeWarps; }

cudaError_t launch_merge(const void* k, const void* v, long long stride_tok, long long stride_head,
                         const Req* reqs, int n_req, int n_kv_heads, long long T,
                         long long total_units, const int* row_ptr, const int* ent_pos,
                         const float* ent_w, const int4* unit_first, int* slot_cnt, float* parts,
                         int varlen_output, long long out_stride_head, void* out_k, void* out_v,
                         int* status, int num_sms, cudaStream_t stream) {
    if (total_units <= 0) return cudaSuccess;
    if (stride_tok <= 0 || stride_tok >= (1ll << 31)) return cudaErrorInvalidValue;   // byte stride kept in 32 bits
    const int smem = (int)sizeof(MergeShared) + 128;
    static unsigned long long configured = 0;
    cudaError_t err = once_per_device(configured, [&]() {
        return cudaFuncSetAttribute(merge_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    });
    if (err != cudaSuccess) return err;
    long long blocks = (total_units + kMergeWarps - 1) / kMergeWarps;
    if (blocks > num_sms) blocks = num_sms;              // persistent: one CTA per SM
    return launch_chained(merge_kernel, dim3((unsigned)blocks), dim3(kMergeWarps * 32), (size_t)smem, stream,
                          (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, stride_tok, stride_head, reqs,
                          n_req, n_kv_heads, T, total_units, row_ptr, ent_pos, ent_w, unit_first, slot_cnt,
                          parts, varlen_output, out_stride_head, (__nv_bfloat16*)out_k, (__nv_bfloat16*)out_v,
                          status);
}

cudaError_t launch_compact_kept(const void* k, const void* v, long long stride_tok,
                                long long stride_head, const Req* reqs, int n_req, int n_kv_heads,
                                long long total_kept_rows, const int* kept_idx, int varlen_output,
                                long long out_stride_head, void* out_k, void* out_v, int* status,
                                cudaStream_t stream) {
    if (total_kept_rows <= 0) return cudaSuccess;
    const long long blocks = (total_kept_rows + 7) / 8;
    return launch_chained(compact_kept_kernel, dim3((unsigned)blocks), dim3(256), 0, stream,
                          (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, stride_tok, stride_head, reqs,
                          n_req, n_kv_heads, total_kept_rows, kept_idx, varlen_output, out_stride_head,
                          (__nv_bfloat16*)out_k, (__nv_bfloat16*)out_v, status);
}

cudaError_t launch_argmax_rows(const float* sim_matrix, const Req* reqs, int n_req,
                                    int n_kv_heads, int max_evicted, int* assign, float* sim,
                                    cudaStream_t stream) {
    if (max_evicted <= 0) return cudaSuccess;
    dim3 grid((max_evicted + 7) / 8, n_kv_heads, n_req);
    argmax_rows_kernel<<<grid, 256, 0, stream>>>(sim_matrix, reqs, n_kv_heads, assign, sim);
    return cudaGetLastError();
}

}  // namespace lookm
