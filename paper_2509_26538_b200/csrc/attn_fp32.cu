// fp32 forward for fp32 inputs: plain FMA arithmetic (no tensor cores, whose
// fp32 modes round operands to tf32 and could not meet a 1e-5 tolerance).
// One warp per query row; every lane runs its own online softmax over the keys
// j = lane, lane + 32, ... of the row's key ranges, and the 32 partial states
// are merged at the end.  Key ranges are those of Algorithm 1: the global prefix
// plus the row's slid tile, or the whole sequence for prefix rows.
#include <math.h>

#include "common.cuh"

namespace hilberta {

constexpr int kRowsPerBlock = 4;

template <int D>
__global__ void __launch_bounds__(kRowsPerBlock * 32)
attn_fp32_kernel(const float *__restrict__ q, const float *__restrict__ k, const float *__restrict__ v,
                 float *__restrict__ out, long long stride_b, long long stride_h, long long stride_s,
                 int heads, int S, int P, const int *__restrict__ row_window,
                 const Window *__restrict__ windows, const int *__restrict__ out_map,
                 const int *__restrict__ in_map, float *__restrict__ lse, float scale) {
    __shared__ float sq[kRowsPerBlock][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * kRowsPerBlock + warp;
    if (row >= S) return;  // whole warp leaves together; no block-wide barrier below
    const int bh = blockIdx.y;
    const long long base = (long long)(bh / heads) * stride_b + (long long)(bh % heads) * stride_h;
    // in_map: q, k, v are in original order and physical row p lives at row in_map[p]
    const float *qrow = q + base + (long long)(in_map ? in_map[row] : row) * stride_s;
    for (int d = lane; d < D; d += 32) sq[warp][d] = qrow[d];
    __syncwarp();

    int seg_start[3], seg_len[3], n_seg;
    const int w = row_window[row];
    if (w < 0) {
        n_seg = 1;
        seg_start[0] = 0;
        seg_len[0] = S;
    } else {
        const Window win = windows[w];
        n_seg = 3;
        seg_start[0] = 0;
        seg_len[0] = P;
        seg_start[1] = win.seg0_start;
        seg_len[1] = win.seg0_len;
        seg_start[2] = win.seg1_start;
        seg_len[2] = win.seg1_len;
    }

    float m = -INFINITY, l = 0.f;
    float acc[D];
#pragma unroll
    for (int d = 0; d < D; ++d) acc[d] = 0.f;

    for (int s = 0; s < n_seg; ++s) {
        const int end = seg_start[s] + seg_len[s];
        for (int j = seg_start[s] + lane; j < end; j += 32) {
            const long long jrow = in_map ? in_map[j] : j;
            const float4 *kj = reinterpret_cast<const float4 *>(k + base + jrow * stride_s);
            float dot = 0.f;
#pragma unroll
            for (int d4 = 0; d4 < D / 4; ++d4) {
                const float4 kk = __ldg(kj + d4);
                dot = fmaf(sq[warp][4 * d4 + 0], kk.x, dot);
                dot = fmaf(sq[warp][4 * d4 + 1], kk.y, dot);
                dot = fmaf(sq[warp][4 * d4 + 2], kk.z, dot);
                dot = fmaf(sq[warp][4 * d4 + 3], kk.w, dot);
            }
            const float x = dot * scale;
            if (x > m) {
                const float corr = expf(m - x);  // exp(-inf) = 0 on the first key
                l *= corr;
#pragma unroll
                for (int d = 0; d < D; ++d) acc[d] *= corr;
                m = x;
            }
            const float p = expf(x - m);
            l += p;
            const float4 *vj = reinterpret_cast<const float4 *>(v + base + jrow * stride_s);
#pragma unroll
            for (int d4 = 0; d4 < D / 4; ++d4) {
                const float4 vv = __ldg(vj + d4);
                acc[4 * d4 + 0] = fmaf(p, vv.x, acc[4 * d4 + 0]);
                acc[4 * d4 + 1] = fmaf(p, vv.y, acc[4 * d4 + 1]);
                acc[4 * d4 + 2] = fmaf(p, vv.z, acc[4 * d4 + 2]);
                acc[4 * d4 + 3] = fmaf(p, vv.w, acc[4 * d4 + 3]);
            }
        }
    }

    // merge the 32 lane states
    float m_all = m;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xffffffffu, m_all, off));
    const float f = (m == -INFINITY) ? 0.f : expf(m - m_all);
    l *= f;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
    const float inv = 1.f / l;
    float mine[D / 32];
#pragma unroll
    for (int d = 0; d < D; ++d) {
        float a = acc[d] * f;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
        if ((d & 31) == lane) mine[d >> 5] = a * inv;
    }
    const int out_row = out_map ? out_map[row] : row;  // optional fused exit scatter
    float *orow = out + base + (long long)out_row * stride_s;
    if (lse && lane == 0) lse[(long long)bh * S + out_row] = m_all + logf(l);
#pragma unroll
    for (int i = 0; i < D / 32; ++i) orow[i * 32 + lane] = mine[i];
}

int launch_attn_fp32(const hilberta_plan_t *p, const void *q, const void *k, const void *v, void *out,
                     float *lse, const int *out_map, const int *in_map, cudaStream_t stream, int chunk) {
    const uintptr_t bits = (uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out;
    if ((bits & 15) || ((p->stride_b | p->stride_h | p->stride_s) & 3)) return HILBERTA_ERR_INVALID;
    int heads = p->heads;
    if (chunk >= 0) {
        // a slice of heads: same strides, shifted base pointers
        if (lse) return HILBERTA_ERR_INVALID;
        heads = p->chunk_heads;
        const long long off = (long long)chunk * heads * p->stride_h;
        q = (const float *)q + off;
        k = (const float *)k + off;
        v = (const float *)v + off;
        out = (float *)out + off;
    }
    dim3 grid((p->S + kRowsPerBlock - 1) / kRowsPerBlock, p->batch * heads);
    dim3 block(kRowsPerBlock * 32);
#define HB_FP32_CASE(DD)                                                                              \
    case DD:                                                                                          \
        attn_fp32_kernel<DD><<<grid, block, 0, stream>>>(                                             \
            (const float *)q, (const float *)k, (const float *)v, (float *)out, p->stride_b,          \
            p->stride_h, p->stride_s, heads, p->S, p->P, p->d_row_window, p->d_windows, out_map, in_map,   \
            lse, p->scale);                                                                                \
        break;
    switch (p->head_dim) {
        HB_FP32_CASE(32)
        HB_FP32_CASE(64)
        HB_FP32_CASE(128)
        default: return HILBERTA_ERR_UNSUPPORTED;
    }
#undef HB_FP32_CASE
    HB_LAUNCHED();
    return HILBERTA_OK;
}

}  // namespace hilberta
