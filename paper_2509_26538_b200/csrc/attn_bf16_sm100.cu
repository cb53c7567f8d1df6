// bf16 block-sparse flash-attention forward for sm_100a (Algorithm 1, restated
// for Blackwell): TMA loads of contiguous Q / K / V tiles, tcgen05 MMAs with
// accumulators in tensor memory, fp32 online softmax, one launch for prefix
// rows and tile rows alike.
//
// A work item is up to 128 consecutive physical query rows that share a key
// list of up to three contiguous ranges (prefix, tile range, wrapped tile
// range -- or the whole sequence for prefix rows).  The key list is cut into
// blocks of 128 keys; the ragged last block of a range is masked by column.
//
// Roles inside a CTA (persistent over work items):
//   warps 0-3  softmax / correction / epilogue, thread r owns query row r
//              (TMEM lane r)
//   warp  4    TMA producer (one elected lane)
//   warp  5    MMA issuer   (one elected lane)
// TMEM columns: [0,128) S = Q K^T (fp32), overwritten in place by P (bf16,
// columns [0,64)); [128,256) O accumulator (fp32).
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <mutex>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace hilberta {
using namespace ptx;

namespace {

constexpr int BM = 128;      // query rows per work item
constexpr int BN = 128;      // keys per block
constexpr int HD = 128;      // head dim
constexpr int STAGES = 2;    // K and V ring depth
constexpr int TILE_BYTES = BN * HD * 2;   // 32 KB: two 64-column slabs of 128 rows
constexpr int SLAB_BYTES = TILE_BYTES / 2;
constexpr int THREADS = 192;
constexpr int SMEM_BYTES = (1 + 2 * STAGES) * TILE_BYTES + 1024;
constexpr uint32_t TMEM_COLS = 256;
constexpr uint32_t TM_S = 0, TM_O = 128;
constexpr long long WAIT_CYCLES = 2000000000ll;  // ~1 s: far beyond any legitimate wait

enum Bar {
    Q_FULL = 0, Q_EMPTY, S_FULL, P_READY, O_DONE, DRAIN,
    K_FULL, K_EMPTY = K_FULL + STAGES, V_FULL = K_EMPTY + STAGES, V_EMPTY = V_FULL + STAGES,
    NUM_BARS = V_EMPTY + STAGES
};

struct Params {
    const WorkItem *work;
    int n_work;
    int bh;      // batch * heads
    int heads;
    long long stride_b, stride_h, stride_s;  // elements
    __nv_bfloat16 *out;
    float scale_log2;
    int *status;
};

// Wait with a deadline; on expiry record where and raise the CTA's abort flag.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                              int *status, int code) {
    const long long t0 = clock64();
    for (uint32_t i = 0;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63) == 63) {
            if (*abort_flag) return false;
            if (clock64() - t0 > WAIT_CYCLES) {
                *abort_flag = 1;
                if (atomicCAS(status, 0, code) == 0) {
                    status[1] = blockIdx.x;
                    status[2] = (int)parity;
                }
                return false;
            }
        }
    }
}

__device__ __forceinline__ int item_blocks(const WorkItem &it, int seg) {
    return (it.seg_len[seg] + BN - 1) / BN;
}

__global__ void __launch_bounds__(THREADS, 1)
attn_bf16_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const Params prm) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[NUM_BARS];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sQ = smem_u32(smem);
    const uint32_t sK = sQ + TILE_BYTES;
    const uint32_t sV = sK + STAGES * TILE_BYTES;
    const int tid = threadIdx.x, warp = tid >> 5;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < NUM_BARS; ++i) mbar_init(bar(i), i == P_READY ? 128 : 1);
        mbar_fence_init();
    }
    if (warp == 4) {
        tmem_alloc(smem_u32(&tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const long long total = (long long)prm.n_work * prm.bh;

    if (warp == 4) {
        // ------------------------------------------------------------ producer
        if (elect_one()) {
            prefetch_tmap(&tmQ);
            prefetch_tmap(&tmK);
            prefetch_tmap(&tmV);
            uint32_t it = 0, qcount = 0;
            bool ok = true;
            for (long long w = blockIdx.x; ok && w < total; w += gridDim.x) {
                const WorkItem wi = prm.work[w / prm.bh];
                const int bh = (int)(w % prm.bh);
                const int b = bh / prm.heads, h = bh % prm.heads;
                ok = wait_or_abort(bar(Q_EMPTY), (qcount & 1) ^ 1, &abort_flag, prm.status, 0x101);
                if (!ok) break;
                mbar_expect_tx(bar(Q_FULL), TILE_BYTES);
                tma_load_4d(sQ, &tmQ, bar(Q_FULL), 0, wi.q_start, h, b);
                tma_load_4d(sQ + SLAB_BYTES, &tmQ, bar(Q_FULL), 64, wi.q_start, h, b);
                ++qcount;
                for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                    const int nb = item_blocks(wi, seg);
                    for (int j = 0; j < nb; ++j, ++it) {
                        const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                        const int row = wi.seg_start[seg] + j * BN;
                        ok = wait_or_abort(bar(K_EMPTY + s), ph ^ 1, &abort_flag, prm.status, 0x102);
                        if (!ok) break;
                        mbar_expect_tx(bar(K_FULL + s), TILE_BYTES);
                        tma_load_4d(sK + s * TILE_BYTES, &tmK, bar(K_FULL + s), 0, row, h, b);
                        tma_load_4d(sK + s * TILE_BYTES + SLAB_BYTES, &tmK, bar(K_FULL + s), 64, row, h, b);
                        ok = wait_or_abort(bar(V_EMPTY + s), ph ^ 1, &abort_flag, prm.status, 0x103);
                        if (!ok) break;
                        mbar_expect_tx(bar(V_FULL + s), TILE_BYTES);
                        tma_load_4d(sV + s * TILE_BYTES, &tmV, bar(V_FULL + s), 0, row, h, b);
                        tma_load_4d(sV + s * TILE_BYTES + SLAB_BYTES, &tmV, bar(V_FULL + s), 64, row, h, b);
                    }
                }
            }
            if (!ok) {
                // let every copy already issued land before the CTA retires
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000) {
                }
            }
        }
    } else if (warp == 5) {
        // ---------------------------------------------------------- MMA issuer
        if (elect_one()) {
            constexpr uint32_t IDESC_QK = idesc_bf16_f32(BM, BN, 0, 0);
            constexpr uint32_t IDESC_PV = idesc_bf16_f32(BM, HD, 0, 1);
            uint32_t it = 0, qcount = 0;
            bool ok = true;
            for (long long w = blockIdx.x; ok && w < total; w += gridDim.x) {
                const WorkItem wi = prm.work[w / prm.bh];
                ok = wait_or_abort(bar(Q_FULL), qcount & 1, &abort_flag, prm.status, 0x201);
                if (!ok) break;
                ++qcount;
                int blk = 0;
                for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                    const int nb = item_blocks(wi, seg);
                    for (int j = 0; j < nb; ++j, ++it, ++blk) {
                        const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                        ok = wait_or_abort(bar(K_FULL + s), ph, &abort_flag, prm.status, 0x202);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll
                        for (int k = 0; k < HD / 16; ++k) {
                            const uint32_t off = (k >> 2) * SLAB_BYTES + (k & 3) * 32;
                            mma_ss(tmem + TM_S, smem_desc_sw128(sQ + off, 16, 1024),
                                   smem_desc_sw128(sK + s * TILE_BYTES + off, 16, 1024), IDESC_QK, k > 0);
                        }
                        mma_commit(bar(K_EMPTY + s));
                        mma_commit(bar(S_FULL));
                        if (blk + 1 == wi.kv_blocks) mma_commit(bar(Q_EMPTY));
                        ok = wait_or_abort(bar(P_READY), it & 1, &abort_flag, prm.status, 0x203);
                        if (!ok) break;
                        ok = wait_or_abort(bar(V_FULL + s), ph, &abort_flag, prm.status, 0x204);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll
                        for (int k = 0; k < BN / 16; ++k) {
                            mma_ts(tmem + TM_O, tmem + TM_S + k * 8,
                                   smem_desc_sw128(sV + s * TILE_BYTES + k * 2048, SLAB_BYTES, 1024), IDESC_PV,
                                   (blk > 0 || k > 0) ? 1u : 0u);
                        }
                        mma_commit(bar(V_EMPTY + s));
                        mma_commit(bar(O_DONE));
                    }
                }
            }
            // every MMA issued above has retired before TMEM is released
            mma_commit(bar(DRAIN));
            wait_or_abort(bar(DRAIN), 0, &abort_flag, prm.status, 0x205);
        }
    } else {
        // ------------------------------------------- softmax / correction / epilogue
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        uint32_t it = 0, ocount = 0;
        bool ok = true;
        for (long long w = blockIdx.x; ok && w < total; w += gridDim.x) {
            const WorkItem wi = prm.work[w / prm.bh];
            const int bh = (int)(w % prm.bh);
            const int b = bh / prm.heads, h = bh % prm.heads;
            float m = -INFINITY, l = 0.f;
            int blk = 0;
            for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                const int nb = item_blocks(wi, seg);
                for (int j = 0; j < nb; ++j, ++it, ++blk) {
                    const int valid = min(BN, wi.seg_len[seg] - j * BN);
                    ok = wait_or_abort(bar(S_FULL), it & 1, &abort_flag, prm.status, 0x301);
                    if (!ok) break;
                    tc_fence_after();
                    float s[BN];
#pragma unroll
                    for (int c = 0; c < BN / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld32(tmem + lane_addr + TM_S + c * 32, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) s[c * 32 + i] = __uint_as_float(r[i]);
                    }
                    float mx = -INFINITY;
#pragma unroll
                    for (int i = 0; i < BN; ++i) {
                        s[i] = (i < valid) ? s[i] * prm.scale_log2 : -INFINITY;
                        mx = fmaxf(mx, s[i]);
                    }
                    const float m_new = fmaxf(m, mx);
                    const float alpha = exp2f(m - m_new);
                    float sum = 0.f;
                    uint32_t pk[BN / 2];
#pragma unroll
                    for (int i = 0; i < BN; i += 2) {
                        const float p0 = exp2f(s[i] - m_new), p1 = exp2f(s[i + 1] - m_new);
                        sum += p0 + p1;
                        __nv_bfloat162 hh = __floats2bfloat162_rn(p0, p1);
                        pk[i >> 1] = *reinterpret_cast<uint32_t *>(&hh);
                    }
                    l = l * alpha + sum;
                    m = m_new;
                    if (blk > 0) {
                        // O accumulated so far belongs to the old maximum
                        ok = wait_or_abort(bar(O_DONE), ocount & 1, &abort_flag, prm.status, 0x302);
                        if (!ok) break;
                        ++ocount;
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < HD / 32; ++c) {
                            uint32_t r[32];
                            tmem_ld32(tmem + lane_addr + TM_O + c * 32, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                            tmem_st32(tmem + lane_addr + TM_O + c * 32, r);
                        }
                    }
#pragma unroll
                    for (int c = 0; c < BN / 64; ++c) {
                        uint32_t r[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = pk[c * 32 + i];
                        tmem_st32(tmem + lane_addr + TM_S + c * 32, r);
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(bar(P_READY));
                }
            }
            if (!ok) break;
            // epilogue: O / l -> bf16 -> global, rows beyond the item are dropped
            ok = wait_or_abort(bar(O_DONE), ocount & 1, &abort_flag, prm.status, 0x303);
            if (!ok) break;
            ++ocount;
            tc_fence_after();
            const float inv = 1.f / l;
            __nv_bfloat16 *orow = prm.out + (long long)b * prm.stride_b + (long long)h * prm.stride_h +
                                  (long long)(wi.q_start + tid) * prm.stride_s;
#pragma unroll
            for (int c = 0; c < HD / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_addr + TM_O + c * 32, r);
                tmem_wait_ld();
                if (tid < wi.q_rows) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint32_t o4[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(r[i + 2 * u]) * inv,
                                                                      __uint_as_float(r[i + 2 * u + 1]) * inv);
                            o4[u] = *reinterpret_cast<uint32_t *>(&hh);
                        }
                        *reinterpret_cast<uint4 *>(orow + c * 32 + i) = make_uint4(o4[0], o4[1], o4[2], o4[3]);
                    }
                }
            }
            tc_fence_before();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        __syncwarp();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

// [batch, heads, S, 128] bf16 with element strides -> 4-D map, box = 64 columns x 128 rows.
int make_map(CUtensorMap *m, const void *base, const hilberta_plan_t *p) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return HILBERTA_ERR_CUDA;
    cuuint64_t dims[4] = {(cuuint64_t)HD, (cuuint64_t)p->S, (cuuint64_t)p->heads, (cuuint64_t)p->batch};
    cuuint64_t strides[3] = {(cuuint64_t)p->stride_s * 2, (cuuint64_t)p->stride_h * 2, (cuuint64_t)p->stride_b * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)BN, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error = (int)cudaErrorInvalidValue;
        return HILBERTA_ERR_CUDA;
    }
    return HILBERTA_OK;
}

void add_items(std::vector<WorkItem> &items, int row0, int rows, int n_seg, const int *seg_start,
               const int *seg_len) {
    for (int r = 0; r < rows; r += BM) {
        WorkItem it{};
        it.q_start = row0 + r;
        it.q_rows = std::min(BM, rows - r);
        it.n_seg = 0;
        it.kv_blocks = 0;
        for (int s = 0; s < n_seg; ++s) {
            if (seg_len[s] <= 0) continue;
            it.seg_start[it.n_seg] = seg_start[s];
            it.seg_len[it.n_seg] = seg_len[s];
            it.kv_blocks += (seg_len[s] + BN - 1) / BN;
            ++it.n_seg;
        }
        items.push_back(it);
    }
}

}  // namespace

// Work list: prefix rows read the whole sequence; the rows of each slid tile
// read the prefix and the tile's own one or two ranges.  Longest items first.
int attn_bf16_prepare(hilberta_plan_t *p) {
    std::vector<WorkItem> items;
    {
        const int st[1] = {0}, ln[1] = {p->S};
        add_items(items, 0, p->P, 1, st, ln);
    }
    for (const Window &w : p->h_windows) {
        const int st[3] = {0, w.seg0_start, w.seg1_start};
        const int ln[3] = {p->P, w.seg0_len, w.seg1_len};
        if (w.seg0_len > 0) add_items(items, w.seg0_start, w.seg0_len, 3, st, ln);
        if (w.seg1_len > 0) add_items(items, w.seg1_start, w.seg1_len, 3, st, ln);
    }
    std::stable_sort(items.begin(), items.end(),
                     [](const WorkItem &a, const WorkItem &b) { return a.kv_blocks > b.kv_blocks; });
    cudaFree(p->d_work);
    p->d_work = nullptr;
    p->n_work = (int)items.size();
    if (items.empty()) return HILBERTA_OK;
    HB_CUDA(cudaMalloc(&p->d_work, sizeof(WorkItem) * items.size()));
    HB_CUDA(cudaMemcpy(p->d_work, items.data(), sizeof(WorkItem) * items.size(), cudaMemcpyHostToDevice));
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(attn_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    });
    HB_CUDA(attr_err);
    return HILBERTA_OK;
}

int launch_attn_bf16(const hilberta_plan_t *p, const void *q, const void *k, const void *v, void *out,
                     cudaStream_t stream) {
    if (p->n_work == 0) return HILBERTA_OK;
    CUtensorMap mq, mk, mv;
    int rc;
    if ((rc = make_map(&mq, q, p)) != HILBERTA_OK) return rc;
    if ((rc = make_map(&mk, k, p)) != HILBERTA_OK) return rc;
    if ((rc = make_map(&mv, v, p)) != HILBERTA_OK) return rc;
    Params prm;
    prm.work = p->d_work;
    prm.n_work = p->n_work;
    prm.bh = p->batch * p->heads;
    prm.heads = p->heads;
    prm.stride_b = p->stride_b;
    prm.stride_h = p->stride_h;
    prm.stride_s = p->stride_s;
    prm.out = (__nv_bfloat16 *)out;
    prm.scale_log2 = p->scale * 1.4426950408889634f;
    prm.status = p->d_status;
    const long long total = (long long)p->n_work * prm.bh;
    const int grid = (int)std::min<long long>(total, p->sm_count);
    attn_bf16_kernel<<<grid, THREADS, SMEM_BYTES, stream>>>(mq, mk, mv, prm);
    HB_LAUNCHED();
    return HILBERTA_OK;
}

}  // namespace hilberta

// Whole path for host-resident activations: H2D copies, three entry gathers,
// forward, exit gather, D2H copy.  Seven device buffers of one tensor each.
extern "C" int hilberta_forward_host(const void *q, const void *k, const void *v, void *out,
                                     hilberta_plan_t *p, void *stream) {
    if (!p || !q || !k || !v || !out) return HILBERTA_ERR_INVALID;
    if (!p->bound) return HILBERTA_ERR_UNBOUND;
    const int64_t dense_h = (int64_t)p->S * p->head_dim;
    if (p->stride_s != p->head_dim || p->stride_h != dense_h || p->stride_b != dense_h * p->heads)
        return HILBERTA_ERR_INVALID;
    const size_t esz = p->dtype == HILBERTA_BF16 ? 2 : 4;
    const size_t bytes = (size_t)p->batch * p->heads * p->S * p->head_dim * esz;
    const size_t slot = (bytes + 255) & ~(size_t)255;
    if (p->ws_bytes < 7 * slot) {
        cudaFree(p->ws);
        p->ws = nullptr;
        p->ws_bytes = 0;
        HB_CUDA(cudaMalloc(&p->ws, 7 * slot));
        p->ws_bytes = 7 * slot;
    }
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = (char *)p->ws;
    void *in[3] = {ws, ws + slot, ws + 2 * slot};
    void *perm[3] = {ws + 3 * slot, ws + 4 * slot, ws + 5 * slot};
    void *out_phys = ws + 6 * slot;
    const void *host_in[3] = {q, k, v};
    const int bh = p->batch * p->heads;
    for (int i = 0; i < 3; ++i) {
        HB_CUDA(cudaMemcpyAsync(in[i], host_in[i], bytes, cudaMemcpyHostToDevice, st));
        int rc = hilberta_permute(in[i], perm[i], p, bh, p->head_dim, p->dtype, st);
        if (rc != HILBERTA_OK) return rc;
    }
    int rc = hilberta_forward(perm[0], perm[1], perm[2], out_phys, p, st);
    if (rc != HILBERTA_OK) return rc;
    rc = hilberta_unpermute(out_phys, in[0], p, bh, p->head_dim, p->dtype, st);
    if (rc != HILBERTA_OK) return rc;
    HB_CUDA(cudaMemcpyAsync(out, in[0], bytes, cudaMemcpyDeviceToHost, st));
    HB_CUDA(cudaStreamSynchronize(st));
    return HILBERTA_OK;
}
