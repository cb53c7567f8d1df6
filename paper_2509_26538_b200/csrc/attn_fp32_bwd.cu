// fp32 backward for fp32 inputs: plain FMA arithmetic, the counterpart of attn_fp32.cu (the
// paper trains through its kernel, Sec. 4.1, without describing the backward pass; this is the
// derivative of Algorithm 1's result).  One warp per resident row; the 32 lanes split the head
// dimension, so every dot product is a warp reduction and every accumulator is D / 32 registers.
//   mode 0: resident = query row i;  for the keys j it sees:  dq_i += dS_ij k_j
//   mode 1: resident = key row j;    for the queries i that see it (the same ranges, the mask
//           being symmetric):  dk_j += dS_ij q_i,  dv_j += P_ij dO_i
// with P_ij = exp(s q_i.k_j - lse_i), dS_ij = P_ij (dO_i.v_j - delta_i).  Not a performance target.
#include <math.h>

#include "common.cuh"

namespace hilberta {

namespace {

constexpr int kRowsPerBlock = 4;

template <int D>
__global__ void __launch_bounds__(kRowsPerBlock * 32)
delta_fp32_kernel(const float *__restrict__ dout, const float *__restrict__ out, float *__restrict__ delta,
                  long long stride_b, long long stride_h, long long stride_s, int heads, int S) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * kRowsPerBlock + warp;
    if (row >= S) return;
    const int bh = blockIdx.y;
    const long long off = (long long)(bh / heads) * stride_b + (long long)(bh % heads) * stride_h +
                          (long long)row * stride_s;
    float acc = 0.f;
#pragma unroll
    for (int e = 0; e < D / 32; ++e) acc = fmaf(dout[off + lane + 32 * e], out[off + lane + 32 * e], acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) delta[(long long)bh * S + row] = acc;
}

template <int D, int MODE>
__global__ void __launch_bounds__(kRowsPerBlock * 32)
attn_fp32_bwd_kernel(const float *__restrict__ q, const float *__restrict__ k, const float *__restrict__ v,
                     const float *__restrict__ dout, const float *__restrict__ lse, const float *__restrict__ delta,
                     float *__restrict__ out_a, float *__restrict__ out_b, long long stride_b, long long stride_h,
                     long long stride_s, int heads, int S, int P, const int *__restrict__ row_window,
                     const Window *__restrict__ windows, float scale) {
    constexpr int E = D / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * kRowsPerBlock + warp;
    if (row >= S) return;
    const int bh = blockIdx.y;
    const long long base = (long long)(bh / heads) * stride_b + (long long)(bh % heads) * stride_h;
    const float *r1 = (MODE == 0 ? q : k) + base + (long long)row * stride_s;
    const float *r2 = (MODE == 0 ? dout : v) + base + (long long)row * stride_s;
    const float *t1 = (MODE == 0 ? k : q) + base;      // streamed operand of the scores
    const float *t2 = (MODE == 0 ? v : dout) + base;   // streamed operand of dP
    float a1[E], a2[E], accA[E], accB[E];
#pragma unroll
    for (int e = 0; e < E; ++e) {
        a1[e] = r1[lane + 32 * e];
        a2[e] = r2[lane + 32 * e];
        accA[e] = 0.f;
        accB[e] = 0.f;
    }
    const float row_lse = lse[(long long)bh * S + row], row_delta = delta[(long long)bh * S + row];

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
    for (int s = 0; s < n_seg; ++s) {
        const int end = seg_start[s] + seg_len[s];
        for (int j = seg_start[s]; j < end; ++j) {
            const float *x1 = t1 + (long long)j * stride_s, *x2 = t2 + (long long)j * stride_s;
            float b1[E], b2[E];
            float dot1 = 0.f, dot2 = 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e) {
                b1[e] = __ldg(x1 + lane + 32 * e);
                b2[e] = __ldg(x2 + lane + 32 * e);
                dot1 = fmaf(a1[e], b1[e], dot1);
                dot2 = fmaf(a2[e], b2[e], dot2);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                dot1 += __shfl_xor_sync(0xffffffffu, dot1, o);
                dot2 += __shfl_xor_sync(0xffffffffu, dot2, o);
            }
            // the statistics belong to the QUERY of the pair
            const float l = MODE == 0 ? row_lse : __ldg(lse + (long long)bh * S + j);
            const float dl = MODE == 0 ? row_delta : __ldg(delta + (long long)bh * S + j);
            const float p = expf(fmaf(dot1, scale, -l));
            const float ds = p * (dot2 - dl);
#pragma unroll
            for (int e = 0; e < E; ++e) {
                accA[e] = fmaf(ds, b1[e], accA[e]);                   // dq += dS k   |  dk += dS q
                if (MODE == 1) accB[e] = fmaf(p, b2[e], accB[e]);     //              |  dv += P dO
            }
        }
    }
    float *oa = out_a + base + (long long)row * stride_s;
#pragma unroll
    for (int e = 0; e < E; ++e) oa[lane + 32 * e] = accA[e] * scale;
    if (MODE == 1) {
        float *ob = out_b + base + (long long)row * stride_s;
#pragma unroll
        for (int e = 0; e < E; ++e) ob[lane + 32 * e] = accB[e];
    }
}

template <int D>
int launch(const hilberta_plan_t *p, const float *dout, const float *q, const float *k, const float *v,
           const float *out, const float *lse, float *dq, float *dk, float *dv, float *delta, cudaStream_t stream) {
    dim3 grid((p->S + kRowsPerBlock - 1) / kRowsPerBlock, p->batch * p->heads);
    dim3 block(kRowsPerBlock * 32);
    delta_fp32_kernel<D><<<grid, block, 0, stream>>>(dout, out, delta, p->stride_b, p->stride_h, p->stride_s, p->heads,
                                                     p->S);
    HB_LAUNCHED();
    attn_fp32_bwd_kernel<D, 0><<<grid, block, 0, stream>>>(q, k, v, dout, lse, delta, dq, nullptr, p->stride_b,
                                                           p->stride_h, p->stride_s, p->heads, p->S, p->P,
                                                           p->d_row_window, p->d_windows, p->scale);
    HB_LAUNCHED();
    attn_fp32_bwd_kernel<D, 1><<<grid, block, 0, stream>>>(q, k, v, dout, lse, delta, dk, dv, p->stride_b,
                                                           p->stride_h, p->stride_s, p->heads, p->S, p->P,
                                                           p->d_row_window, p->d_windows, p->scale);
    HB_LAUNCHED();
    return HILBERTA_OK;
}

}  // namespace

int launch_attn_fp32_bwd(const hilberta_plan_t *p, const void *dout, const void *q, const void *k, const void *v,
                         const void *out, const float *lse, void *dq, void *dk, void *dv, float *delta,
                         cudaStream_t stream) {
    if ((p->stride_b | p->stride_h | p->stride_s) & 3) return HILBERTA_ERR_INVALID;
    switch (p->head_dim) {
        case 32:
            return launch<32>(p, (const float *)dout, (const float *)q, (const float *)k, (const float *)v,
                              (const float *)out, lse, (float *)dq, (float *)dk, (float *)dv, delta, stream);
        case 64:
            return launch<64>(p, (const float *)dout, (const float *)q, (const float *)k, (const float *)v,
                              (const float *)out, lse, (float *)dq, (float *)dk, (float *)dv, delta, stream);
        case 128:
            return launch<128>(p, (const float *)dout, (const float *)q, (const float *)k, (const float *)v,
                               (const float *)out, lse, (float *)dq, (float *)dk, (float *)dv, delta, stream);
        default: return HILBERTA_ERR_UNSUPPORTED;
    }
}

}  // namespace hilberta
