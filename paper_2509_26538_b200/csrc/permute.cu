// Entry / exit row gathers of Sec. 3.4: HBM-bound copies of whole token rows
// through an index table.  Both directions are written as gathers (reads are
// indirect, writes are sequential), with 16-byte accesses and four independent
// loads in flight per thread; the grid covers the tensor in one pass.
#include "common.cuh"

namespace hilberta {

constexpr int kGatherThreads = 256;
constexpr int kGatherUnroll = 4;

// dst[b, r, :] = src[b, index[r], :]; a row is `vecs` 16-byte vectors.
__global__ void __launch_bounds__(kGatherThreads)
row_gather_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, const int *__restrict__ index,
                  int rows, int vecs, long long total) {
    const long long stride = (long long)gridDim.x * kGatherThreads;
    long long g = (long long)blockIdx.x * kGatherThreads + threadIdx.x;
    const long long per_batch = (long long)rows * vecs;
    for (; g < total; g += stride * kGatherUnroll) {
        uint4 val[kGatherUnroll];
        long long at[kGatherUnroll];
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u) {
            const long long e = g + (long long)u * stride;
            at[u] = e;
            if (e < total) {
                const long long b = e / per_batch;
                const long long rem = e - b * per_batch;
                const int r = (int)(rem / vecs);
                const int c = (int)(rem - (long long)r * vecs);
                const int s = __ldg(index + r);
                val[u] = __ldcs(src + b * per_batch + (long long)s * vecs + c);
            }
        }
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u)
            if (at[u] < total) __stcs(dst + at[u], val[u]);
    }
}

static int gather(const void *src, void *dst, const int *index, const hilberta_plan_t *p, int batch,
                  int row_elems, int dtype, cudaStream_t stream) {
    if (!p || !src || !dst || batch < 1 || row_elems < 1) return HILBERTA_ERR_INVALID;
    if (dtype != HILBERTA_BF16 && dtype != HILBERTA_FP32 && dtype != HILBERTA_FP8_E4M3) return HILBERTA_ERR_INVALID;
    int dev = -1;
    HB_CUDA(cudaGetDevice(&dev));
    if (dev != p->device) return HILBERTA_ERR_INVALID;  // the plan's tables live on another device
    const size_t esz = dtype == HILBERTA_BF16 ? 2 : dtype == HILBERTA_FP8_E4M3 ? 1 : 4;
    const size_t row_bytes = (size_t)row_elems * esz;
    if (row_bytes % 16 || ((uintptr_t)src & 15) || ((uintptr_t)dst & 15)) return HILBERTA_ERR_INVALID;
    const size_t bytes = row_bytes * (size_t)p->S * (size_t)batch;
    const char *a = (const char *)src, *b = (const char *)dst;
    if (a < b + bytes && b < a + bytes) return HILBERTA_ERR_INVALID;  // overlap
    const int vecs = (int)(row_bytes / 16);
    const long long total = (long long)batch * p->S * vecs;
    long long blocks = (total + (long long)kGatherThreads * kGatherUnroll - 1) /
                       ((long long)kGatherThreads * kGatherUnroll);
    // One pass per thread (four independent 16-byte copies) measured fastest: a capped grid whose
    // threads loop a second, partly filled time lost 20 % of the copy bandwidth.
    const long long cap = 0x7fffffffll;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    row_gather_kernel<<<(unsigned)blocks, kGatherThreads, 0, stream>>>(
        (const uint4 *)src, (uint4 *)dst, index, p->S, vecs, total);
    HB_LAUNCHED();
    return HILBERTA_OK;
}

}  // namespace hilberta

extern "C" int hilberta_permute(const void *src, void *dst, const hilberta_plan_t *plan, int batch,
                                int row_elems, int dtype, void *stream) {
    return hilberta::gather(src, dst, plan ? plan->d_phys2orig : nullptr, plan, batch, row_elems, dtype,
                            (cudaStream_t)stream);
}

extern "C" int hilberta_unpermute(const void *src, void *dst, const hilberta_plan_t *plan, int batch,
                                  int row_elems, int dtype, void *stream) {
    return hilberta::gather(src, dst, plan ? plan->d_orig2phys : nullptr, plan, batch, row_elems, dtype,
                            (cudaStream_t)stream);
}
