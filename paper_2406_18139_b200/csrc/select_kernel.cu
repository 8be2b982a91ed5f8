// Selection kernel: recent window, text prior and Top-N (Eq. 5-8), one CTA per (request, KV head).
//
// The text prior is applied as an ordering rule: adding T_p = max(A_s) to every text score makes
// any text token outrank any image token (scores are positive), so candidates are ordered by
// (is_text, score, lower position).  With n_text text candidates and N slots:
//   n_text <= N : all text candidates are kept and the best N - n_text image candidates;
//   n_text >  N : the best N text candidates are kept and no image candidate.
// Without a mask (text prior off: Eq. 8 on the raw scores) every candidate is in the text class,
// which reduces to a plain Top-N by score.
// Either way one class is kept wholesale or not at all and the other needs an exact top-k, done
// by a 4-pass radix select on an order-preserving 32-bit key; ties at the threshold go to the
// lowest positions.  A final ordered pass writes the kept and evicted lists in ascending position.
//
// The selection occupies only n_requests * n_kv_heads CTAs, so the same launch carries, in further
// CTAs, work that does not depend on it and is needed next: 1 / |k| of every key row (the cosine
// denominators of Eq. 9).
#include <cuda_bf16.h>

#include <algorithm>

#include "internal.h"

namespace lookm {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kPerThread = 8;
constexpr int kKeyCache = 8;                         // candidates per thread whose keys stay in registers

__device__ __forceinline__ unsigned order_key(float s) {
    unsigned b = __float_as_uint(s);
    if (b == 0x80000000u) b = 0u;                        // -0 and +0 compare equal
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);   // larger float <=> larger key
}

// Exclusive block scan of two ints per thread; returns the block totals through ta / tb.
__device__ __forceinline__ void block_scan2(int a, int b, int& ea, int& eb, int& ta, int& tb,
                                            int (*warp_tot)[2]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int ia = a, ib = b;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int xa = __shfl_up_sync(0xffffffffu, ia, o);
        const int xb = __shfl_up_sync(0xffffffffu, ib, o);
        if (lane >= o) { ia += xa; ib += xb; }
    }
    __syncthreads();                                     // protects warp_tot from the previous use
    if (lane == 31) { warp_tot[warp][0] = ia; warp_tot[warp][1] = ib; }
    __syncthreads();
    if (warp == 0) {
        int wa = warp_tot[lane][0], wb = warp_tot[lane][1];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int xa = __shfl_up_sync(0xffffffffu, wa, o);
            const int xb = __shfl_up_sync(0xffffffffu, wb, o);
            if (lane >= o) { wa += xa; wb += xb; }
        }
        warp_tot[lane][0] = wa;
        warp_tot[lane][1] = wb;
    }
    __syncthreads();
    const int ba = warp ? warp_tot[warp - 1][0] : 0;
    const int bb = warp ? warp_tot[warp - 1][1] : 0;
    ea = ba + ia - a;
    eb = bb + ib - b;
    ta = warp_tot[31][0];
    tb = warp_tot[31][1];
}

// 1 / |k| of every key row (0 for a zero row): half a warp per row, 16 bytes per lane, four rows
// in flight per half-warp (the loop is bound by memory latency otherwise).  Row r is token
// r / n_kv_heads of head r % n_kv_heads; the quotient and remainder are carried along instead of
// divided out every time.
__device__ __forceinline__ void key_norms(const __nv_bfloat16* __restrict__ k, long long stride_tok,
                                          long long stride_head, int n_kv_heads, long long T,
                                          float* __restrict__ rnorm_all, int block, int n_blocks) {
    constexpr int kRowsPerBlock = kSelThreads / 16;
    constexpr int kFlight = 4;
    const int half = threadIdx.x >> 4, l16 = threadIdx.x & 15;
    const long long n_rows = T * n_kv_heads;
    const long long step = (long long)n_blocks * kRowsPerBlock;      // rows between two of my rows
    const long long step_tok = step / n_kv_heads;
    const int step_h = (int)(step % n_kv_heads);
    long long r = (long long)block * kRowsPerBlock + half;
    long long tok = r / n_kv_heads;
    int h = (int)(r % n_kv_heads);
    // the loop bound is the warp's first row, so that both half-warps always reach the shuffles
    for (long long rw = r - (half & 1); rw < n_rows; rw += kFlight * step) {
        uint4 u[kFlight];
        long long tok_i[kFlight];
        int h_i[kFlight];
        bool valid[kFlight];
#pragma unroll
        for (int i = 0; i < kFlight; ++i) {
            valid[i] = r < n_rows;
            tok_i[i] = tok;
            h_i[i] = h;
            u[i] = make_uint4(0u, 0u, 0u, 0u);
            if (valid[i]) u[i] = *reinterpret_cast<const uint4*>(k + tok * stride_tok + h * stride_head + l16 * 8);
            r += step;
            tok += step_tok;
            h += step_h;
            if (h >= n_kv_heads) { h -= n_kv_heads; ++tok; }
        }
#pragma unroll
        for (int i = 0; i < kFlight; ++i) {
            const unsigned w[4] = {u[i].x, u[i].y, u[i].z, u[i].w};
            float ss = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float lo = __uint_as_float(w[j] << 16), hi = __uint_as_float(w[j] & 0xffff0000u);
                ss = fmaf(lo, lo, ss);
                ss = fmaf(hi, hi, ss);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o, 16);
            if (l16 == 0 && valid[i]) rnorm_all[(long long)h_i[i] * T + tok_i[i]] = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
        }
    }
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, const uint8_t* __restrict__ mask,
              const Req* __restrict__ reqs, int n_select_blocks, int n_kv_heads, long long T,
              int* __restrict__ kept_idx, int* __restrict__ evict_idx, int* __restrict__ rank,
              const __nv_bfloat16* __restrict__ keys, long long stride_tok, long long stride_head,
              float* __restrict__ rnorm_all) {
    __shared__ int hist[256];
    __shared__ int warp_tot[32][2];
    __shared__ int sh_val[4];

    grid_dependency_wait();
    if ((int)blockIdx.x >= n_select_blocks) {
        key_norms(keys, stride_tok, stride_head, n_kv_heads, T, rnorm_all, (int)blockIdx.x - n_select_blocks,
                  (int)gridDim.x - n_select_blocks);
        return;
    }
    const Req rq = reqs[blockIdx.x / n_kv_heads];
    const int h = blockIdx.x % n_kv_heads;
    const float* s = scores + (long long)h * T + rq.tok_begin;
    const uint8_t* msk = mask ? mask + rq.tok_begin : nullptr;
    auto is_image = [msk](int j) { return msk != nullptr && msk[j] != 0; };
    const int L = rq.L, B = rq.B, M = rq.M;
    const int N = B - M, nc = L - M;

    // ---- count text candidates; the first kKeyCache * 1024 candidates' keys and classes stay in
    // registers for the radix passes (the loads would otherwise be repeated in every pass, and
    // each round trip is paid in full by this latency-bound kernel) -----------------------------
    int cnt = 0;
    unsigned ckey[kKeyCache];
    unsigned cimg = 0u;                                  // bit q: cached candidate q is an image token
#pragma unroll
    for (int q = 0; q < kKeyCache; ++q) {
        const int j = threadIdx.x + q * kSelThreads;
        ckey[q] = 0u;
        if (j < nc) {
            const bool img = is_image(j);
            ckey[q] = order_key(s[j]);
            cimg |= (img ? 1u : 0u) << q;
            cnt += !img;
        }
    }
    for (int j = threadIdx.x + kKeyCache * kSelThreads; j < nc; j += kSelThreads) cnt += !is_image(j);
    {
        int e0, e1, t0, t1;
        block_scan2(cnt, 0, e0, e1, t0, t1, warp_tot);
        cnt = t0;
    }
    const int n_text = cnt;
    // class whose members are ranked (1 = image); the other class is kept entirely or not at all
    const int sel_cls = (n_text <= N) ? 1 : 0;
    const bool other_kept = (n_text <= N);
    int k = (n_text <= N) ? (N - n_text) : N;            // how many of sel_cls to keep
    const int n_sel = sel_cls ? (nc - n_text) : n_text;

    // ---- radix select: key of the k-th largest member of sel_cls -------------------------------
    unsigned thr = 0u;          // threshold key
    int need_ties = 0;          // members equal to thr to keep (lowest positions first)
    bool take_all = (k >= n_sel), take_none = (k <= 0);
    if (!take_all && !take_none) {
        unsigned prefix = 0u, pmask = 0u;
        int remaining = k;
        for (int shift = 24; shift >= 0; shift -= 8) {
            for (int i = threadIdx.x; i < 256; i += kSelThreads) hist[i] = 0;
            __syncthreads();
#pragma unroll
            for (int q = 0; q < kKeyCache; ++q) {
                const int j = threadIdx.x + q * kSelThreads;
                if (j < nc && ((cimg >> q) & 1u) == (unsigned)sel_cls && (ckey[q] & pmask) == prefix)
                    atomicAdd(&hist[(ckey[q] >> shift) & 255u], 1);
            }
            for (int j = threadIdx.x + kKeyCache * kSelThreads; j < nc; j += kSelThreads) {
                if (is_image(j) == (sel_cls != 0)) {
                    const unsigned key = order_key(s[j]);
                    if ((key & pmask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
                }
            }
            __syncthreads();
            if (threadIdx.x < 32) {
                // digit d with (count of digits above d) < remaining <= (count of digits >= d):
                // lane l owns the digits 255 - 8l .. 248 - 8l, scanned from the top
                const int lane = threadIdx.x;
                int c[8], mine = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) { c[q] = hist[255 - 8 * lane - q]; mine += c[q]; }
                int incl = mine;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int x = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += x;
                }
                const unsigned reach = __ballot_sync(0xffffffffu, incl >= remaining);
                const int owner = reach ? __ffs(reach) - 1 : 31;      // reach is never 0: k <= n_sel
                if (lane == owner) {
                    int acc = incl - mine, q = 0;
                    for (; q < 7; ++q) {
                        if (acc + c[q] >= remaining) break;
                        acc += c[q];
                    }
                    sh_val[0] = 255 - 8 * lane - q;
                    sh_val[1] = remaining - acc;             // still to take inside that digit
                }
            }
            __syncthreads();
            prefix |= (unsigned)sh_val[0] << shift;
            pmask |= 255u << shift;
            remaining = sh_val[1];
            __syncthreads();
        }
        thr = prefix;
        need_ties = remaining;
    }

    // ---- ordered emission -----------------------------------------------------------------------
    const long long kept_base = rq.kept_off + (long long)h * B;
    const long long ev_base = rq.ev_off + (long long)h * rq.E;
    int* rk = rank ? rank + (long long)h * T + rq.tok_begin : nullptr;
    int kept_run = 0, tie_run = 0;
    for (int base = 0; base < L; base += kSelThreads * kPerThread) {
        const int j0 = base + threadIdx.x * kPerThread;
        int keep[kPerThread], tie[kPerThread];
        int nk = 0, nt = 0;
#pragma unroll
        for (int q = 0; q < kPerThread; ++q) {
            const int j = j0 + q;
            keep[q] = 0;
            tie[q] = 0;
            if (j < L) {
                if (j >= nc) {
                    keep[q] = 1;
                } else {
                    const int cls = is_image(j);
                    if (cls != sel_cls) {
                        keep[q] = other_kept;
                    } else if (take_all) {
                        keep[q] = 1;
                    } else if (!take_none) {
                        const unsigned key = order_key(s[j]);
                        if (key > thr) keep[q] = 1;
                        else if (key == thr) tie[q] = 1;
                    }
                }
            }
            nt += tie[q];
        }
        // ties first: a tie is kept while fewer than need_ties equal keys precede it
        int e_tie, e_dummy, t_tie, t_dummy;
        block_scan2(nt, 0, e_tie, e_dummy, t_tie, t_dummy, warp_tot);
        int tr = tie_run + e_tie;
#pragma unroll
        for (int q = 0; q < kPerThread; ++q) {
            if (tie[q]) { if (tr < need_ties) keep[q] = 1; ++tr; }
            nk += keep[q];
        }
        int e_keep, t_keep;
        block_scan2(nk, 0, e_keep, e_dummy, t_keep, t_dummy, warp_tot);
        int slot = kept_run + e_keep;
#pragma unroll
        for (int q = 0; q < kPerThread; ++q) {
            const int j = j0 + q;
            if (j < L) {
                if (keep[q]) {
                    kept_idx[kept_base + slot] = j;
                    if (rk) rk[j] = -1 - slot;
                    ++slot;
                } else {
                    const int e = j - slot;              // evicted before j = j - kept before j
                    evict_idx[ev_base + e] = j;
                    if (rk) rk[j] = e;
                }
            }
        }
        kept_run += t_keep;
        tie_run += t_tie;
    }
}

}  // namespace

cudaError_t launch_select(const float* scores, const uint8_t* mask, const Req* reqs, int n_req,
                          int n_kv_heads, long long T, int* kept_idx, int* evict_idx, int* rank,
                          const void* k_for_norms, long long stride_tok, long long stride_head,
                          float* rnorm_all, int num_sms, cudaStream_t stream) {
    const int n_select = n_kv_heads * n_req;
    int n_norm = 0;
    if (k_for_norms) {
        // one CTA of this kernel fits on an SM: the norm CTAs take the SMs that the selection
        // leaves free, so that all of them run at once (a second wave would have to wait for the
        // selection CTAs, which run longest)
        const long long want = (T * n_kv_heads + kSelThreads / 16 - 1) / (kSelThreads / 16);
        // (with selection CTAs on more than half of the SMs the few SMs left would carry all the
        // norms: then a full wave of norm CTAs follows the selection CTAs instead)
        n_norm = (int)std::min<long long>(want, n_select < num_sms / 2 ? num_sms - n_select : num_sms);
    }
    return launch_chained(select_kernel, dim3(n_select + n_norm), dim3(kSelThreads), 0, stream,
                          scores, mask, reqs, n_select, n_kv_heads, T, kept_idx, evict_idx, rank,
                          (const __nv_bfloat16*)k_for_norms, stride_tok, stride_head, rnorm_all);
}

}  // namespace lookm
