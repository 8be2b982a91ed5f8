// The step after the compression path: one token-generation step of one layer over a (compressed)
// KV cache (Section 3.1, Eq. 2-3).  The new token's K and V rows are appended to the cache and
// every query head attends over its KV head's rows, the new one included:
//     out_g = softmax(q_g K^T * scale) V.
//
// The step is bound by HBM bandwidth: every cached K and V row (256 bytes each) is read exactly
// once per step, whatever the number of query heads in the group, and nothing else of any size
// moves.  The rows of a (request, KV head) are cut into splits of `rows_per_split` rows (chosen
// per call so that the grid fills the GPU a few times over); a CTA of 8 warps takes one split:
// half a warp owns a row (16 bytes per lane), four rows per half-warp are in flight at a time, the
// dot products are reduced with four shuffles, and each half-warp keeps its own running softmax
// statistics (reference maximum, sum, weighted V sum) for every query head of the group in
// registers.  Half-warps and warps are combined through shared memory in a fixed order; with more
// than one split the CTA leaves its partial result in the workspace and the CTA that arrives last
// at the (request, KV head) adds the splits in split order.  No CTA waits for another and the
// order of additions never depends on timing, so results are reproducible bit for bit.
#include <cuda_bf16.h>
#include <math.h>

#include "internal.h"

namespace lookm {
namespace {

constexpr int kDecThreads = 256;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kDecHalfWarps = 2 * kDecWarps;         // rows a CTA has in hand at once
constexpr int kDecFlight = 4;                        // rows in flight per half-warp

__device__ __forceinline__ void unpack_bf16x8(const uint4& u, float (&x)[8]) {
    const unsigned w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

__device__ __forceinline__ float dec_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int GT>
struct DecShared {
    float m[kDecWarps][GT];                          // [warp][query head of the pass]
    float l[kDecWarps][GT];
    float o[kDecWarps][GT][kHeadDim];
    int last;
};

// GT query heads of the group are handled per pass over the rows (GT divides the group size).
template <int GT>
__global__ void __launch_bounds__(kDecThreads)
decode_kernel(const __grid_constant__ DecodeBatch batch, const __nv_bfloat16* __restrict__ q,
              const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new,
              __nv_bfloat16* __restrict__ cache_k, __nv_bfloat16* __restrict__ cache_v,
              long long stride_row, long long stride_head, int n_q_heads, int n_kv_heads, int group,
              int rows_per_split, float scale_log2, float* __restrict__ parts, int* __restrict__ arrivals,
              float* __restrict__ out) {
    __shared__ DecShared<GT> sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hw = threadIdx.x >> 4, l16 = lane & 15;

    // which (request, KV head, pass, split) this CTA owns: requests are found by their first CTA
    int r = 0;
    {
        int lo = 0, hi = batch.n_req - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (batch.r[mid].cta_begin <= (int)blockIdx.x) lo = mid; else hi = mid - 1;
        }
        r = lo;
    }
    const DecodeReq rq = batch.r[r];
    const int n_pass = group / GT;
    const int local = (int)blockIdx.x - rq.cta_begin;            // [head][pass][split]
    const int split = local % rq.n_splits;
    const int pass = (local / rq.n_splits) % n_pass;
    const int h = local / (rq.n_splits * n_pass);
    const int n_rows = rq.len + 1;                               // cached rows + the new one
    const int row0 = split * rows_per_split, row1 = min(n_rows, row0 + rows_per_split);
    const int qh0 = h * group + pass * GT;                       // first query head of this pass

    grid_dependency_wait();

    // this lane's 8 features of the GT query rows
    float qv[GT][8];
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        const uint4 u = *reinterpret_cast<const uint4*>(q + ((long long)rq.index * n_q_heads + qh0 + g) * kHeadDim + l16 * 8);
        unpack_bf16x8(u, qv[g]);
    }
    const long long head_off = (long long)h * stride_head + l16 * 8;
    const __nv_bfloat16* ck = cache_k + rq.begin * stride_row + head_off;
    const __nv_bfloat16* cv = cache_v + rq.begin * stride_row + head_off;
    const __nv_bfloat16* nk = k_new + ((long long)rq.index * n_kv_heads + h) * kHeadDim + l16 * 8;
    const __nv_bfloat16* nv = v_new + ((long long)rq.index * n_kv_heads + h) * kHeadDim + l16 * 8;

    float m[GT], l[GT], o[GT][8];
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        m[g] = -INFINITY;
        l[g] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) o[g][i] = 0.f;
    }

    // the loop bound does not depend on the half-warp, so both halves of a warp reach the shuffles
    for (int base = row0; base < row1; base += kDecHalfWarps * kDecFlight) {
        uint4 ku[kDecFlight], vu[kDecFlight];
        bool valid[kDecFlight];
#pragma unroll
        for (int f = 0; f < kDecFlight; ++f) {
            const int row = base + f * kDecHalfWarps + hw;
            valid[f] = row < row1;
            ku[f] = make_uint4(0u, 0u, 0u, 0u);
            vu[f] = make_uint4(0u, 0u, 0u, 0u);
            if (valid[f]) {
                const bool is_new = (row == rq.len);             // Eq. 2: the appended row
                const __nv_bfloat16* kp = is_new ? nk : ck + (long long)row * stride_row;
                const __nv_bfloat16* vp = is_new ? nv : cv + (long long)row * stride_row;
                ku[f] = __ldg(reinterpret_cast<const uint4*>(kp));
                vu[f] = __ldg(reinterpret_cast<const uint4*>(vp));
                if (is_new && pass == 0) {                       // the cache grows by this row
                    *reinterpret_cast<uint4*>(cache_k + rq.begin * stride_row + head_off + (long long)row * stride_row) = ku[f];
                    *reinterpret_cast<uint4*>(cache_v + rq.begin * stride_row + head_off + (long long)row * stride_row) = vu[f];
                }
            }
        }
        float s[kDecFlight][GT];
#pragma unroll
        for (int f = 0; f < kDecFlight; ++f) {
            float kx[8];
            unpack_bf16x8(ku[f], kx);
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                float d = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) d = fmaf(qv[g][i], kx[i], d);
#pragma unroll
                for (int ofs = 8; ofs > 0; ofs >>= 1) d += __shfl_xor_sync(0xffffffffu, d, ofs, 16);
                s[f][g] = valid[f] ? d : -INFINITY;
            }
        }
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            float mx = m[g];
#pragma unroll
            for (int f = 0; f < kDecFlight; ++f) mx = fmaxf(mx, s[f][g]);
            if (mx == -INFINITY) continue;                       // no valid row for this half-warp yet
            const float alpha = dec_ex2((m[g] - mx) * scale_log2);   // 0 when m was -inf
            float p[kDecFlight], ps = 0.f;
#pragma unroll
            for (int f = 0; f < kDecFlight; ++f) {
                p[f] = dec_ex2((s[f][g] - mx) * scale_log2);     // 0 for an invalid row
                ps += p[f];
            }
            l[g] = l[g] * alpha + ps;
            m[g] = mx;
#pragma unroll
            for (int i = 0; i < 8; ++i) o[g][i] *= alpha;
#pragma unroll
            for (int f = 0; f < kDecFlight; ++f) {
                float vx[8];
                unpack_bf16x8(vu[f], vx);
#pragma unroll
                for (int i = 0; i < 8; ++i) o[g][i] = fmaf(p[f], vx[i], o[g][i]);
            }
        }
    }

    // ---- combine: the two half-warps of a warp in registers, then the warps in warp order -------
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        const float m_o = __shfl_xor_sync(0xffffffffu, m[g], 16);
        const float l_o = __shfl_xor_sync(0xffffffffu, l[g], 16);
        const float mx = fmaxf(m[g], m_o);
        // lower half-warp first, whichever half this lane is in
        const bool low = lane < 16;
        const float a_me = (mx == -INFINITY) ? 0.f : dec_ex2((m[g] - mx) * scale_log2);
        const float a_ot = (mx == -INFINITY) ? 0.f : dec_ex2((m_o - mx) * scale_log2);
        const float l_lo = low ? l[g] * a_me : l_o * a_ot, l_hi = low ? l_o * a_ot : l[g] * a_me;
        l[g] = l_lo + l_hi;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float o_o = __shfl_xor_sync(0xffffffffu, o[g][i], 16);
            const float o_lo = low ? o[g][i] * a_me : o_o * a_ot, o_hi = low ? o_o * a_ot : o[g][i] * a_me;
            o[g][i] = o_lo + o_hi;
        }
        m[g] = mx;
        if (lane == 0) { sh.m[warp][g] = m[g]; sh.l[warp][g] = l[g]; }
        if (low) {
#pragma unroll
            for (int i = 0; i < 8; ++i) sh.o[warp][g][l16 * 8 + i] = o[g][i];
        }
    }
    __syncthreads();
    // thread t < 128 owns feature t of every query head of the pass
    const int n_splits = rq.n_splits;
    const long long part_stride = kHeadDim + 2;                  // m, l, o[128]
    float* my_parts = parts + ((long long)rq.part_begin + ((long long)(h * n_pass + pass) * n_splits + split) * GT) * part_stride;
    if (threadIdx.x < kHeadDim) {
        const int t = threadIdx.x;
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            float mx = -INFINITY;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) mx = fmaxf(mx, sh.m[w][g]);
            float lsum = 0.f, osum = 0.f;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) {
                const float a = dec_ex2((sh.m[w][g] - mx) * scale_log2);   // 0 for an idle warp
                lsum = fmaf(sh.l[w][g], a, lsum);
                osum = fmaf(sh.o[w][g][t], a, osum);
            }
            if (n_splits == 1) {
                out[((long long)rq.index * n_q_heads + qh0 + g) * kHeadDim + t] = osum / lsum;
            } else {
                float* rec = my_parts + g * part_stride;
                if (t == 0) { rec[0] = mx; rec[1] = lsum; }
                rec[2 + t] = osum;
            }
        }
    }
    if (n_splits == 1) return;

    // ---- several splits: the CTA that arrives last adds them in split order ----------------------
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        int* cnt = arrivals + rq.arrival_begin + h * n_pass + pass;
        const int prev = atomicAdd(cnt, 1);
        sh.last = (prev == n_splits - 1);
        if (sh.last) *cnt = 0;                                   // ready for the next step
    }
    __syncthreads();
    if (!sh.last) return;
    __threadfence();
    if (threadIdx.x < kHeadDim) {
        const int t = threadIdx.x;
        const float* base = parts + ((long long)rq.part_begin + (long long)(h * n_pass + pass) * n_splits * GT) * part_stride;
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            float mx = -INFINITY;
            for (int sp = 0; sp < n_splits; ++sp) mx = fmaxf(mx, __ldcg(base + ((long long)sp * GT + g) * part_stride));
            float lsum = 0.f, osum = 0.f;
            for (int sp = 0; sp < n_splits; ++sp) {
                const float* rec = base + ((long long)sp * GT + g) * part_stride;
                const float a = dec_ex2((__ldcg(rec) - mx) * scale_log2);
                lsum = fmaf(__ldcg(rec + 1), a, lsum);
                osum = fmaf(__ldcg(rec + 2 + t), a, osum);
            }
            out[((long long)rq.index * n_q_heads + qh0 + g) * kHeadDim + t] = osum / lsum;
        }
    }
}

}  // namespace

cudaError_t launch_decode(const DecodeBatch& batch, int total_ctas, int gt, const void* q,
                          const void* k_new, const void* v_new, void* cache_k, void* cache_v,
                          long long stride_row, long long stride_head, int n_q_heads, int n_kv_heads,
                          int rows_per_split, float scale_log2, float* parts, int* arrivals,
                          float* out, cudaStream_t stream) {
    if (total_ctas <= 0) return cudaSuccess;
    const int group = n_q_heads / n_kv_heads;
#define LOOKM_LAUNCH_DECODE(GT)                                                                     \
    return launch_chained(decode_kernel<GT>, dim3((unsigned)total_ctas), dim3(kDecThreads), 0, stream, \
                          batch, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k_new,              \
                          (const __nv_bfloat16*)v_new, (__nv_bfloat16*)cache_k, (__nv_bfloat16*)cache_v, \
                          stride_row, stride_head, n_q_heads, n_kv_heads, group, rows_per_split,    \
                          scale_log2, parts, arrivals, out);
    if (gt == 8) { LOOKM_LAUNCH_DECODE(8) }
    if (gt == 4) { LOOKM_LAUNCH_DECODE(4) }
    if (gt == 2) { LOOKM_LAUNCH_DECODE(2) }
    LOOKM_LAUNCH_DECODE(1)
#undef LOOKM_LAUNCH_DECODE
}

}  // namespace lookm
