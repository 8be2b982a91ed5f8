// The step after the compression path: one token-generation step of one layer over a (compressed)
// KV cache (Section 3.1, Eq. 2-3).  The new token's K and V rows are appended to the cache and
// every query head attends over its KV head's rows, the new one included:
//     out_g = softmax(q_g K^T * scale) V.
//
// The step is bound by HBM bandwidth: every cached K and V row (256 bytes each) is read exactly
// once per step, whatever the number of query heads in the group, and nothing else of any size
// moves.  The rows of a (request, KV head) are cut into splits of `rows_per_split` rows (chosen
// per call so that the grid is one wave of resident CTAs); a CTA of 8 warps takes one split: half a
// warp owns a row (16 bytes per lane).  Rows travel global -> shared memory with 16-byte cp.async
// copies into a ring private to each warp (a step = four K and four V rows per half-warp; the
// steps ahead are in flight while one is worked on, and every lane reads back exactly the bytes it
// copied, so cp.async.wait_group is all the synchronisation there is).  The dot products are
// reduced with four shuffles, and each half-warp keeps its own running softmax statistics
// (reference maximum, sum, weighted V sum) for every query head of the group in registers.  Half-warps and warps are combined through shared memory in a fixed order; with more
// than one split the CTA leaves its partial result in the workspace and a second kernel, chained
// behind the first, adds the splits in split order.  No CTA waits for another and the order of
// additions never depends on timing, so results are reproducible bit for bit.
#include <cuda_bf16.h>
#include <math.h>

#include "internal.h"

namespace lookm {
namespace {

constexpr int kDecThreads = kDecodeThreads;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kDecHalfWarps = 2 * kDecWarps;         // rows a CTA has in hand at once
#ifndef LOOKM_DEC_FLIGHT
#define LOOKM_DEC_FLIGHT 4
#endif
#ifndef LOOKM_DEC_RING
#define LOOKM_DEC_RING 4
#endif
constexpr int kDecFlight = LOOKM_DEC_FLIGHT;         // rows per half-warp and step
constexpr int kDecRing = LOOKM_DEC_RING;             // steps in the ring of a warp (all but one in flight)
constexpr int kDecRowBytes = kHeadDim * 2;
constexpr int kDecStepBytes = 2 * kDecFlight * 2 * kDecRowBytes;   // per warp: [half][row][K|V][256 B]
constexpr int kDecRingBytes = kDecWarps * kDecRing * kDecStepBytes;

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
};

// GT query heads of the group are handled per pass over the rows (GT divides the group size).
template <int GT>
__global__ void __launch_bounds__(kDecThreads)
decode_kernel(const __grid_constant__ DecodeBatch batch, const __nv_bfloat16* __restrict__ q,
              const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new,
              __nv_bfloat16* __restrict__ cache_k, __nv_bfloat16* __restrict__ cache_v,
              long long stride_row, long long stride_head, int n_q_heads, int n_kv_heads, int group,
              int rows_per_split, float scale_log2, float* __restrict__ parts, float* __restrict__ out) {
    __shared__ DecShared<GT> sh;
    extern __shared__ __align__(128) uint8_t dec_ring[];         // [warp][ring step][half][row][K|V][256 B]
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

    // The appended row (Eq. 2) is read from k_new / v_new by whoever owns it; the CTA that owns it
    // on the group's first pass also writes it into the cache (nobody reads cache row `len` in this
    // step, so the write races with nothing).
    if (pass == 0 && rq.len >= row0 && rq.len < row1 && warp == 0) {
        const __nv_bfloat16* src = lane < 16 ? nk : nv;
        __nv_bfloat16* dst = (lane < 16 ? cache_k : cache_v) + rq.begin * stride_row + head_off +
                             (long long)rq.len * stride_row;
        *reinterpret_cast<uint4*>(dst) = __ldg(reinterpret_cast<const uint4*>(src));
    }

    // Copies of one step: K and V of kDecFlight rows per half-warp, 16 bytes per lane and row,
    // straight into this warp's ring.  Rows past the split are zero-filled (a copy of 0 source
    // bytes), so that they contribute exact zeros.  One commit group per step, also past the end.
    const uint32_t ring0 = (uint32_t)__cvta_generic_to_shared(dec_ring) + warp * (kDecRing * kDecStepBytes) +
                           ((lane >> 4) * kDecFlight * 2) * kDecRowBytes + l16 * 16;
    auto issue = [&](int step) {
        const int base = row0 + step * (kDecHalfWarps * kDecFlight);
        const uint32_t dst = ring0 + (uint32_t)(step % kDecRing) * kDecStepBytes;
        if (base < row1) {
#pragma unroll
            for (int f = 0; f < kDecFlight; ++f) {
                const int row = base + f * kDecHalfWarps + hw;
                const bool is_new = (row == rq.len);
                const bool valid = row < row1;
                const __nv_bfloat16* kp = (is_new || !valid) ? nk : ck + (long long)row * stride_row;
                const __nv_bfloat16* vp = (is_new || !valid) ? nv : cv + (long long)row * stride_row;
                const int nbytes = valid ? 16 : 0;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                             ::"r"(dst + (2 * f) * kDecRowBytes), "l"(kp), "r"(nbytes) : "memory");
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                             ::"r"(dst + (2 * f + 1) * kDecRowBytes), "l"(vp), "r"(nbytes) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // Softmax statistics and weighted V sums of one step's rows (online softmax against the running
    // maximum of this half-warp).
    auto consume = [&](int step) {
        const int base = row0 + step * (kDecHalfWarps * kDecFlight);
        const uint32_t src = ring0 + (uint32_t)(step % kDecRing) * kDecStepBytes;
        uint4 ku[kDecFlight], vu[kDecFlight];
#pragma unroll
        for (int f = 0; f < kDecFlight; ++f) {
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(ku[f].x), "=r"(ku[f].y), "=r"(ku[f].z), "=r"(ku[f].w)
                         : "r"(src + (2 * f) * kDecRowBytes));
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(vu[f].x), "=r"(vu[f].y), "=r"(vu[f].z), "=r"(vu[f].w)
                         : "r"(src + (2 * f + 1) * kDecRowBytes));
        }
        float s[kDecFlight][GT];
#pragma unroll
        for (int f = 0; f < kDecFlight; ++f) {
            const bool valid = base + f * kDecHalfWarps + hw < row1;
            float kx[8];
            unpack_bf16x8(ku[f], kx);
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                float d = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) d = fmaf(qv[g][i], kx[i], d);
#pragma unroll
                for (int ofs = 8; ofs > 0; ofs >>= 1) d += __shfl_xor_sync(0xffffffffu, d, ofs, 16);
                s[f][g] = valid ? d : -INFINITY;
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
    };

    // the step count does not depend on the half-warp, so both halves of a warp reach the shuffles
    const int n_steps = (row1 - row0 + kDecHalfWarps * kDecFlight - 1) / (kDecHalfWarps * kDecFlight);
#pragma unroll
    for (int st = 0; st < kDecRing - 1; ++st) issue(st);
    for (int st = 0; st < n_steps; ++st) {
        // the buffer refilled here was read into registers one iteration ago
        issue(st + kDecRing - 1);
        asm volatile("cp.async.wait_group %0;" ::"n"(kDecRing - 1) : "memory");
        consume(st);
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
}

// Several splits: adds the partial results of one (request, KV head, pass, query head) in split
// order.  One CTA of 128 threads per such unit, thread t owns feature t; the splits' reference
// values are fetched in one round trip and the records of sixteen splits are requested together
// (the kernel is bound by the latency of these loads).  Launched
// behind decode_kernel with programmatic stream serialisation: no counters, no atomics, nothing in
// the workspace has to be cleared, and the order of additions is fixed.
__global__ void __launch_bounds__(kHeadDim)
decode_combine_kernel(const __grid_constant__ DecodeBatch batch, int gt, int n_pass, int n_q_heads, int group,
                      float scale_log2, const float* __restrict__ parts, float* __restrict__ out) {
    const DecodeReq rq = batch.r[blockIdx.y];
    const int n_splits = rq.n_splits;
    const int g = (int)blockIdx.x % gt, unit = (int)blockIdx.x / gt;     // unit = h * n_pass + pass
    const int pass = unit % n_pass, h = unit / n_pass;
    const int t = threadIdx.x;
    grid_dependency_wait();
    if (n_splits == 1) return;                                   // decode_kernel wrote the output itself
    const long long part_stride = kHeadDim + 2;
    const float* base = parts + ((long long)rq.part_begin + (long long)unit * n_splits * gt + g) * part_stride;
    const long long step = (long long)gt * part_stride;          // between the records of two splits
    // largest reference value over the splits: thread t looks at splits t, t + 128, ...; one round
    // trip for up to 128 splits, then a block-wide maximum
    __shared__ float warp_max[kHeadDim / 32];
    float mx = -INFINITY;
    for (int sp = t; sp < n_splits; sp += kHeadDim) mx = fmaxf(mx, __ldcg(base + sp * step));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if ((t & 31) == 0) warp_max[t >> 5] = mx;
    __syncthreads();
    mx = fmaxf(fmaxf(warp_max[0], warp_max[1]), fmaxf(warp_max[2], warp_max[3]));
    // the records in split order, kBatch of them requested together
    constexpr int kBatch = 16;
    float lsum = 0.f, osum = 0.f;
    for (int s0 = 0; s0 < n_splits; s0 += kBatch) {
        float mv[kBatch], lv[kBatch], ov[kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const bool in = s0 + j < n_splits;
            const float* rec = base + (s0 + j) * step;
            mv[j] = in ? __ldcg(rec) : -INFINITY;
            lv[j] = in ? __ldcg(rec + 1) : 0.f;
            ov[j] = in ? __ldcg(rec + 2 + t) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const float a = dec_ex2((mv[j] - mx) * scale_log2);  // 0 past the last split
            lsum = fmaf(lv[j], a, lsum);
            osum = fmaf(ov[j], a, osum);
        }
    }
    out[((long long)rq.index * n_q_heads + h * group + pass * gt + g) * kHeadDim + t] = osum / lsum;
}

}  // namespace

// The ring needs more dynamic shared memory than the default limit: raised once per device.
static cudaError_t configure_decode() {
    static unsigned long long configured = 0;
    return once_per_device(configured, []() {
        cudaError_t e = cudaFuncSetAttribute(decode_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecRingBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecRingBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecRingBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecRingBytes);
        return e;
    });
}

// CTAs of decode_kernel<gt> that one SM holds at a time on the current device (looked up once per
// device); 0 if the query fails.  The planner sizes the grid to one such wave.
int decode_ctas_per_sm(int gt) {
    static int cache[64][4] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    const int idx = gt == 8 ? 3 : gt == 4 ? 2 : gt == 2 ? 1 : 0;
    int v = __atomic_load_n(&cache[dev][idx], __ATOMIC_ACQUIRE);
    if (v > 0) return v;
    if (configure_decode() != cudaSuccess) { cudaGetLastError(); return 0; }
    cudaError_t err;
    if (idx == 3) err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, decode_kernel<8>, kDecThreads, kDecRingBytes);
    else if (idx == 2) err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, decode_kernel<4>, kDecThreads, kDecRingBytes);
    else if (idx == 1) err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, decode_kernel<2>, kDecThreads, kDecRingBytes);
    else err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, decode_kernel<1>, kDecThreads, kDecRingBytes);
    if (err != cudaSuccess || v <= 0) { cudaGetLastError(); return 0; }
    __atomic_store_n(&cache[dev][idx], v, __ATOMIC_RELEASE);
    return v;
}

cudaError_t launch_decode(const DecodeBatch& batch, int total_ctas, int gt, const void* q,
                          const void* k_new, const void* v_new, void* cache_k, void* cache_v,
                          long long stride_row, long long stride_head, int n_q_heads, int n_kv_heads,
                          int rows_per_split, float scale_log2, float* parts, float* out,
                          cudaStream_t stream) {
    if (total_ctas <= 0) return cudaSuccess;
    const int group = n_q_heads / n_kv_heads;
    cudaError_t err = configure_decode();
    if (err != cudaSuccess) return err;
#define LOOKM_LAUNCH_DECODE(GT)                                                                     \
    err = launch_chained(decode_kernel<GT>, dim3((unsigned)total_ctas), dim3(kDecThreads),          \
                         (size_t)kDecRingBytes, stream,                                             \
                         batch, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k_new,               \
                         (const __nv_bfloat16*)v_new, (__nv_bfloat16*)cache_k, (__nv_bfloat16*)cache_v, \
                         stride_row, stride_head, n_q_heads, n_kv_heads, group, rows_per_split,     \
                         scale_log2, parts, out);
    if (gt == 8) { LOOKM_LAUNCH_DECODE(8) }
    else if (gt == 4) { LOOKM_LAUNCH_DECODE(4) }
    else if (gt == 2) { LOOKM_LAUNCH_DECODE(2) }
    else { LOOKM_LAUNCH_DECODE(1) }
#undef LOOKM_LAUNCH_DECODE
    return err;
}

cudaError_t launch_decode_combine(const DecodeBatch& batch, int gt, int n_q_heads, int n_kv_heads,
                                  float scale_log2, const float* parts, float* out, cudaStream_t stream) {
    const int group = n_q_heads / n_kv_heads;
    const int n_pass = group / gt;
    return launch_chained(decode_combine_kernel, dim3((unsigned)(n_kv_heads * n_pass * gt), (unsigned)batch.n_req),
                          dim3(kHeadDim), 0, stream, batch, gt, n_pass, n_q_heads, group, scale_log2, parts, out);
}

}  // namespace lookm
