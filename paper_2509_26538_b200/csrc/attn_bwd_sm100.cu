// bf16 backward pass of the block-sparse attention for sm_100a.  The paper trains
// through its kernel (Sec. 4.1) without describing the backward pass; this is the
// derivative of Algorithm 1's result on the same physical layout, key lists and
// work items as the forward kernel (the mask is symmetric, so the queries that see
// a key tile are listed exactly like the keys a query tile sees).
//
// With P = exp(s Q K^T - LSE), dP = dO V^T, delta = rowsum(dO * O) and
// dS = P * (dP - delta):   dQ = s dS K,   dK = s dS^T Q,   dV = P^T dO.
//
// Three launches: a bandwidth-bound pass that writes delta, then one tensor-core
// kernel in two modes that share all code but the element-wise step.
//   mode DQ : resident tile = 128 query rows (Q_i, dO_i); streamed = their keys (K_j, V_j)
//             acc1 = Q_i K_j^T, acc2 = dO_i V_j^T, dS -> TMEM, dQ_i += dS K_j
//   mode DKV: resident tile = 128 key rows (K_j, V_j); streamed = the queries that see them
//             acc1 = K_j Q_i^T, acc2 = V_j dO_i^T (transposed scores: a thread owns a KEY row),
//             P^T, dS^T -> TMEM, dV_j += P^T dO_i, dK_j += dS^T Q_i
// Streamed rows come in sub-blocks of 64 with two accumulator buffers, so the MMAs of
// sub-block s + 1 run while the CUDA cores work on sub-block s; the two element-wise
// warpgroups each take 32 of the 64 columns of every sub-block, which halves the
// latency of the MMA -> element-wise -> MMA chain.  TMEM: acc1/acc2 of buffer b at
// [128 b, +64) and [128 b + 64, +64); P and dS (bf16) overwrite them in place, each
// warpgroup inside the columns it has just read.  DKV: two buffers, dK at [256, 384),
// dV at [384, 512).  DQ: three buffers (the MMAs run two sub-blocks ahead), dQ at [384, 512).
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <functional>
#include <mutex>
#include <queue>
#include <utility>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace hilberta {
using namespace ptx;

int make_tensor_map(CUtensorMap *m, const void *base, const hilberta_plan_t *p, int box_rows);

namespace {

constexpr int BM = 128;   // resident rows per work item
constexpr int SUB = 64;   // streamed rows per sub-block
constexpr int HD = 128;
constexpr int NST_MAX = 5;   // ring of streamed sub-blocks (two 16-KB tiles each): 5 slots in DQ mode, 4 in DKV
#ifndef HB_NST_DQ
#define HB_NST_DQ 5
#endif
#ifndef HB_NST_DKV
#define HB_NST_DKV 4
#endif
__host__ __device__ constexpr int nst_of(int mode) { return mode == 0 ? HB_NST_DQ : HB_NST_DKV; }
constexpr int RES_BYTES = BM * HD * 2;        // 32 KB: two 64-column slabs of 128 rows
constexpr int RES_SLAB = RES_BYTES / 2;
constexpr int SUBT_BYTES = SUB * HD * 2;      // 16 KB: two 64-column slabs of 64 rows
constexpr int SUBT_SLAB = SUBT_BYTES / 2;
constexpr int STAGE_BYTES = 2 * SUBT_BYTES;
constexpr int THREADS = 512;  // 8 element-wise warps, 4 single-lane service warps, 4 epilogue warps
// accumulator buffers: DQ has TMEM for three (its output needs 128 columns), DKV for two
__host__ __device__ constexpr int nb_of(int mode) { return mode == 0 ? 3 : 2; }
__host__ __device__ constexpr int smem_bytes_of(int mode) { return 2 * RES_BYTES + nst_of(mode) * STAGE_BYTES + 1024; }
constexpr uint32_t TMEM_COLS = 512;
constexpr int MODE_DQ = 0, MODE_DKV = 1;

enum Bar {
    RES_FULL = 0, RES_EMPTY, OUT_FULL, EPI_DONE, DRAIN,
    S_FULL,                      // [NB] acc1 / acc2 of buffer b written
    P_READY = S_FULL + 3,        // [NB] P / dS of buffer b written, 256 arrivals
    ST_FULL = P_READY + 3, ST_EMPTY = ST_FULL + NST_MAX,
    STAT_FULL = ST_EMPTY + NST_MAX,   // DKV: statistics of the streamed rows of ring slot s written
    NUM_BARS = STAT_FULL + NST_MAX
};

struct Params {
    const WorkItem *work;
    const WorkUnit *units;
    const int *cta_begin;
    int heads;
    long long stride_b, stride_h, stride_s;  // elements
    const float *lse;     // [batch * heads, S], natural log
    const float *delta;   // [batch * heads, S]
    __nv_bfloat16 *out_a; // DQ: dq; DKV: dk
    __nv_bfloat16 *out_b; // DKV: dv
    float scale, scale_log2;
    int S;
    int out_align32;      // outputs and strides 32-byte aligned: 32-byte stores allowed
    int *status;
};

__device__ __forceinline__ int sub_blocks(const WorkItem &it, int seg) {
    return (it.seg_len[seg] + SUB - 1) / SUB;
}

// acc = R T^T: resident tile (128 rows) times a streamed sub-block (64 rows), K = head dim.
__device__ __forceinline__ void issue_rt(uint32_t tmem_acc, uint32_t sR, uint32_t sT) {
    constexpr uint32_t IDESC = idesc_bf16_f32(BM, SUB, 0, 0);
    const uint64_t da = smem_desc_sw128(sR, 16, 1024), db = smem_desc_sw128(sT, 16, 1024);
#pragma unroll
    for (int k = 0; k < HD / 16; ++k) {
        const uint64_t oa = (uint64_t)(((k >> 2) * RES_SLAB + (k & 3) * 32) >> 4);
        const uint64_t ob = (uint64_t)(((k >> 2) * SUBT_SLAB + (k & 3) * 32) >> 4);
        mma_ss(tmem_acc, da + oa, db + ob, IDESC, k > 0);
    }
}

// out (+)= A T: A (128 x 64, bf16) from TMEM, the streamed sub-block row-major in smem
// (N-major operand: 64 rows of K, two 64-column slabs of N).
// A sits where each element-wise warpgroup left it: the bf16 pairs of streamed rows
// [32 w, 32 w + 32) occupy columns [32 w, 32 w + 16) of the fp32 block they were computed from.
__device__ __forceinline__ void issue_at(uint32_t tmem_out, uint32_t tmem_a, uint32_t sT, bool accumulate) {
    constexpr uint32_t IDESC = idesc_bf16_f32(BM, HD, 0, 1);
    const uint64_t db = smem_desc_sw128(sT, SUBT_SLAB, 1024);
#pragma unroll
    for (int k = 0; k < SUB / 16; ++k)
        mma_ts(tmem_out, tmem_a + (k >> 1) * 32 + (k & 1) * 8, db + (uint64_t)((k * 2048) >> 4), IDESC,
               (accumulate || k > 0) ? 1u : 0u);
}

template <int MODE>
__global__ void __launch_bounds__(THREADS, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmR1, const __grid_constant__ CUtensorMap tmR2,
                const __grid_constant__ CUtensorMap tmT1, const __grid_constant__ CUtensorMap tmT2,
                const Params prm) {
    constexpr int NST = nst_of(MODE);
    constexpr int NB = nb_of(MODE), LA = NB - 1;          // MMAs run LA sub-blocks ahead of the element-wise step
    constexpr uint32_t OUT_A = MODE == MODE_DKV ? 256 : 384, OUT_B = 384;  // TMEM columns of the outputs
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[NUM_BARS];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ __align__(16) float stats[MODE == MODE_DKV ? NST : 1][2][SUB];  // DKV: lse (base 2), delta of streamed rows

    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sR1 = smem_u32(smem), sR2 = sR1 + RES_BYTES;
    const uint32_t sST = sR2 + RES_BYTES;
    const int tid = threadIdx.x, warp = tid >> 5;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < NUM_BARS; ++i) {
            uint32_t count = 1;
            if (i == EPI_DONE) count = 128;
            if (i >= P_READY && i < P_READY + 3) count = 256;
            mbar_init(bar(i), count);
        }
        mbar_fence_init();
    }
    if (warp == 8) {
        tmem_alloc(smem_u32(&tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const int u_begin = prm.cta_begin[blockIdx.x], u_end = prm.cta_begin[blockIdx.x + 1];

    if (warp >= 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
    }
    if (warp == 8) {
        // ------------------------------------------------ producer of the streamed sub-blocks
        if (elect_one()) {
            prefetch_tmap(&tmT1);
            prefetch_tmap(&tmT2);
            uint32_t g = 0;
            bool ok = true;
            for (int u = u_begin; ok && u < u_end; ++u) {
                const WorkUnit unit = prm.units[u];
                const WorkItem wi = prm.work[unit.item];
                const int b = unit.bh / prm.heads, h = unit.bh % prm.heads;
                for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                    const int nb = sub_blocks(wi, seg);
                    for (int j = 0; j < nb; ++j, ++g) {
                        const int row = wi.seg_start[seg] + j * SUB;
                        const uint32_t s = g % NST, ph = (g / NST) & 1;
                        ok = wait_or_abort(bar(ST_EMPTY + s), ph ^ 1, &abort_flag, prm.status, 0x402);
                        if (!ok) break;
                        const uint32_t dst = sST + s * STAGE_BYTES;
                        mbar_expect_tx(bar(ST_FULL + s), STAGE_BYTES);
                        tma_load_4d(dst, &tmT1, bar(ST_FULL + s), 0, row, h, b);
                        tma_load_4d(dst + SUBT_SLAB, &tmT1, bar(ST_FULL + s), 64, row, h, b);
                        tma_load_4d(dst + SUBT_BYTES, &tmT2, bar(ST_FULL + s), 0, row, h, b);
                        tma_load_4d(dst + SUBT_BYTES + SUBT_SLAB, &tmT2, bar(ST_FULL + s), 64, row, h, b);
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
    } else if (warp == 10) {
        // ------------------------------------------------ loader of the resident tiles
        // A thread of its own, so that the sub-block producer can run ahead into the next unit
        // while this one waits for the resident tiles to be released.
        if (elect_one()) {
            prefetch_tmap(&tmR1);
            prefetch_tmap(&tmR2);
            uint32_t uc = 0;
            bool ok = true;
            for (int u = u_begin; ok && u < u_end; ++u, ++uc) {
                const WorkUnit unit = prm.units[u];
                const WorkItem wi = prm.work[unit.item];
                const int b = unit.bh / prm.heads, h = unit.bh % prm.heads;
                // free once the last R T^T MMA of the previous unit has retired
                if (uc > 0) ok = wait_or_abort(bar(RES_EMPTY), (uc - 1) & 1, &abort_flag, prm.status, 0x401);
                if (!ok) break;
                mbar_expect_tx(bar(RES_FULL), 2 * RES_BYTES);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t off = (i >> 1) * RES_SLAB + (i & 1) * (SUB * 128);
                    tma_load_4d(sR1 + off, &tmR1, bar(RES_FULL), (i >> 1) * 64, wi.q_start + (i & 1) * SUB, h, b);
                    tma_load_4d(sR2 + off, &tmR2, bar(RES_FULL), (i >> 1) * 64, wi.q_start + (i & 1) * SUB, h, b);
                }
                if (u + 1 < u_end) {
                    // pull the next unit's resident tiles into L2 while this unit runs
                    const WorkUnit nu = prm.units[u + 1];
                    const int nq = prm.work[nu.item].q_start;
                    const int nb_ = nu.bh / prm.heads, nh = nu.bh % prm.heads;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        tma_prefetch_4d(&tmR1, (i >> 1) * 64, nq + (i & 1) * SUB, nh, nb_);
                        tma_prefetch_4d(&tmR2, (i >> 1) * 64, nq + (i & 1) * SUB, nh, nb_);
                    }
                }
            }
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000) {
                }
            }
        }
    } else if (warp == 11) {
        // ------------------------------------------------ DKV: statistics of the streamed query rows
        // lse (base 2) and delta of the 64 rows of every sub-block go to shared memory, two
        // sub-blocks ahead of use; rows beyond the range get lse = +inf, which turns their
        // weights into exact zeros.
        if (MODE == MODE_DKV) {
            const int lane = tid & 31;
            struct It {
                int u, seg, j, bh;
                WorkItem wi;
                bool valid;
            };
            auto load_unit = [&](It &it) {
                it.valid = it.u < u_end;
                if (it.valid) {
                    const WorkUnit unit = prm.units[it.u];
                    it.wi = prm.work[unit.item];
                    it.bh = unit.bh;
                }
            };
            auto advance = [&](It &it) {
                if (++it.j >= sub_blocks(it.wi, it.seg)) {
                    it.j = 0;
                    if (++it.seg >= it.wi.n_seg) {
                        it.seg = 0;
                        ++it.u;
                        load_unit(it);
                    }
                }
            };
            auto fetch = [&](const It &it, float (&l2)[2], float (&dl)[2]) {
                if (!it.valid) return;
                const int row = it.wi.seg_start[it.seg] + it.j * SUB;
                const int valid = min(SUB, it.wi.seg_len[it.seg] - it.j * SUB);
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int c = lane + 32 * i;
                    l2[i] = __int_as_float(0x7f800000);
                    dl[i] = 0.f;
                    if (c < valid) {
                        l2[i] = __ldg(prm.lse + (long long)it.bh * prm.S + row + c) * 1.4426950408889634f;
                        dl[i] = __ldg(prm.delta + (long long)it.bh * prm.S + row + c);
                    }
                }
            };
            uint32_t g = 0;
            bool ok = true;
            auto publish = [&](const float (&l2)[2], const float (&dl)[2]) {
                const uint32_t s = g % NST, ph = (g / NST) & 1;
                if (lane == 0) ok = wait_or_abort(bar(ST_EMPTY + s), ph ^ 1, &abort_flag, prm.status, 0x701);
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) return;
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    stats[s][0][lane + 32 * i] = l2[i];
                    stats[s][1][lane + 32 * i] = dl[i];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(STAT_FULL + s));
                ++g;
            };
            It cur{u_begin, 0, 0, 0, WorkItem{}, false}, pre{u_begin, 0, 0, 0, WorkItem{}, false};
            load_unit(cur);
            load_unit(pre);
            float al2[2], adl[2], bl2[2], bdl[2];
            fetch(pre, al2, adl);
            if (pre.valid) advance(pre);
            fetch(pre, bl2, bdl);
            if (pre.valid) advance(pre);
            while (ok && cur.valid) {
                publish(al2, adl);
                if (!ok) break;
                advance(cur);
                fetch(pre, al2, adl);
                if (pre.valid) advance(pre);
                if (!cur.valid) break;
                publish(bl2, bdl);
                if (!ok) break;
                advance(cur);
                fetch(pre, bl2, bdl);
                if (pre.valid) advance(pre);
            }
        }
    } else if (warp >= 12) {
        // ------------------------------------------------ epilogue: accumulators -> bf16 -> global
        // Its own warpgroup, so that the element-wise warps move on to the next unit at once.
        const int r = tid & 127;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        uint32_t uc = 0;
        bool ok = true;
        for (int u = u_begin; ok && u < u_end; ++u, ++uc) {
            const WorkUnit unit = prm.units[u];
            const WorkItem wi = prm.work[unit.item];
            const int b = unit.bh / prm.heads, h = unit.bh % prm.heads;
            const bool row_ok = r < wi.q_rows;
            ok = wait_or_abort(bar(OUT_FULL), uc & 1, &abort_flag, prm.status, 0x605);
            if (!ok) break;
            tc_fence_after();
            const long long roff = (long long)b * prm.stride_b + (long long)h * prm.stride_h +
                                   (long long)(wi.q_start + r) * prm.stride_s;
            constexpr int NCH = (MODE == MODE_DKV) ? 8 : 4;   // DKV: dK then dV
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                uint32_t o[32];
                tmem_ld32(tmem + lane_addr + OUT_A + c * 32, o);
                tmem_wait_ld();
                if (row_ok) {
                    __nv_bfloat16 *orow = (c >= 4 ? prm.out_b : prm.out_a) + roff + (c & 3) * 32;
                    const float mul = c >= 4 ? 1.f : prm.scale;
                    uint32_t w[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        w[i] = pack_bf16(__uint_as_float(o[2 * i]) * mul, __uint_as_float(o[2 * i + 1]) * mul);
                    if (prm.out_align32) {
                        st_global_v8(orow, w);
                        st_global_v8(orow + 16, w + 8);
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; i += 4)
                            *reinterpret_cast<uint4 *>(orow + 2 * i) = make_uint4(w[i], w[i + 1], w[i + 2], w[i + 3]);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bar(EPI_DONE));
        }
    } else if (warp == 9) {
        // ---------------------------------------------------------- MMA issuer
        if (elect_one()) {
            uint32_t g = 0, uc = 0;
            uint32_t cP[3] = {0, 0, 0};
            bool ok = true;
#ifdef HB_BWD_TIMING
            long long tw_res = 0, tw_st = 0, tw_epi = 0, tw_p = 0, tw_st0 = 0, tw_p0 = 0, t_mark, t_start = clock64();
#define TMARK() t_mark = clock64()
#define TACC(x) x += clock64() - t_mark
#else
#define TMARK()
#define TACC(x)
#endif
            for (int u = u_begin; ok && u < u_end; ++u, ++uc) {
                const WorkItem wi = prm.work[prm.units[u].item];
                const int n = wi.kv_blocks;  // sub-blocks of this item
                TMARK();
                ok = wait_or_abort(bar(RES_FULL), uc & 1, &abort_flag, prm.status, 0x501);
                TACC(tw_res);
                if (!ok) break;
                for (int s = 0; s < n + LA; ++s) {
                    if (s < n) {
                        const uint32_t e = g + s, slot = e % NST;
                        TMARK();
                        ok = wait_or_abort(bar(ST_FULL + slot), (e / NST) & 1, &abort_flag, prm.status, 0x502);
                        TACC(tw_st);
#ifdef HB_BWD_TIMING
                        if (s < 2) tw_st0 += clock64() - t_mark;
#endif
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t sT = sST + slot * STAGE_BYTES;
                        const uint32_t acc = tmem + (s % NB) * 128;
                        issue_rt(acc, sR1, sT);
                        issue_rt(acc + 64, sR2, sT + SUBT_BYTES);
                        mma_commit(bar(S_FULL + (s % NB)));
                        if (s == n - 1) mma_commit(bar(RES_EMPTY));
                    }
                    if (s >= LA) {
                        const int sp = s - LA, bf = sp % NB;
                        const uint32_t e = g + sp, slot = e % NST;
                        if (sp == 0 && uc > 0) {
                            // the previous unit's accumulators have been read out
                            TMARK();
                            ok = wait_or_abort(bar(EPI_DONE), (uc - 1) & 1, &abort_flag, prm.status, 0x503);
                            TACC(tw_epi);
                            if (!ok) break;
                        }
                        TMARK();
                        ok = wait_or_abort(bar(P_READY + bf), cP[bf] & 1, &abort_flag, prm.status, 0x504 + bf);
                        TACC(tw_p);
#ifdef HB_BWD_TIMING
                        if (sp < 2) tw_p0 += clock64() - t_mark;
#endif
                        if (!ok) break;
                        ++cP[bf];
                        tc_fence_after();
                        const uint32_t sT = sST + slot * STAGE_BYTES;
                        const uint32_t acc = tmem + bf * 128;
                        issue_at(tmem + OUT_A, acc + 64, sT, sp > 0);                                  // dS  x T1
                        if (MODE == MODE_DKV) issue_at(tmem + OUT_B, acc, sT + SUBT_BYTES, sp > 0);  // P^T x T2
                        mma_commit(bar(ST_EMPTY + slot));
                    }
                }
                if (!ok) break;
                mma_commit(bar(OUT_FULL));
                g += n;
            }
            // every MMA issued above has retired before TMEM is released
            mma_commit(bar(DRAIN));
            wait_or_abort(bar(DRAIN), 0, &abort_flag, prm.status, 0x507);
#ifdef HB_BWD_TIMING
            atomicAdd(prm.status + 32 + MODE * 8 + 0, (int)(tw_res >> 6));
            atomicAdd(prm.status + 32 + MODE * 8 + 1, (int)(tw_st >> 6));
            atomicAdd(prm.status + 32 + MODE * 8 + 2, (int)(tw_epi >> 6));
            atomicAdd(prm.status + 32 + MODE * 8 + 3, (int)(tw_p >> 6));
            atomicAdd(prm.status + 32 + MODE * 8 + 4, (int)((clock64() - t_start) >> 6));
            atomicMax(prm.status + 32 + MODE * 8 + 5, (int)((clock64() - t_start) >> 6));
            atomicAdd(prm.status + 32 + MODE * 8 + 6, (int)(tw_st0 >> 6));
            atomicAdd(prm.status + 32 + MODE * 8 + 7, (int)(tw_p0 >> 6));
#endif
        }
    } else if (warp < 8) {
        // ------------------------------------ element-wise step + epilogue, warpgroup wg
        asm volatile("setmaxnreg.inc.sync.aligned.u32 168;");
        const int wg = warp >> 2;
        const int r = tid & 127;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const float scale_log2 = prm.scale_log2;
        uint32_t cS[3] = {0, 0, 0}, g = 0, uc = 0;
        bool ok = true;
        for (int u = u_begin; ok && u < u_end; ++u, ++uc) {
            const WorkUnit unit = prm.units[u];
            const WorkItem wi = prm.work[unit.item];
            const int bh = unit.bh;
            const int b = bh / prm.heads, h = bh % prm.heads;
            const bool row_ok = r < wi.q_rows;
            // DQ: this thread's query row statistics
            float row_l2 = __int_as_float(0x7f800000), row_dl = 0.f;
            if (MODE == MODE_DQ && row_ok) {
                row_l2 = prm.lse[(long long)bh * prm.S + wi.q_start + r] * 1.4426950408889634f;
                row_dl = prm.delta[(long long)bh * prm.S + wi.q_start + r];
            }
            int s = 0;
            for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                const int nb = sub_blocks(wi, seg);
                for (int j = 0; j < nb; ++j, ++s) {
                    const int bf = s % NB;
                    // this warpgroup's 32 columns of the sub-block
                    const int valid = min(SUB, wi.seg_len[seg] - j * SUB) - wg * 32;
                    const uint32_t tAcc = tmem + lane_addr + bf * 128;
                    const uint32_t e = g + s, slot = e % NST;
                    if (MODE == MODE_DKV) {
                        ok = wait_or_abort(bar(STAT_FULL + slot), (e / NST) & 1, &abort_flag, prm.status, 0x601 + wg);
                        if (!ok) break;
                    }
                    ok = wait_or_abort(bar(S_FULL + bf), cS[bf] & 1, &abort_flag, prm.status, 0x603 + wg);
                    if (!ok) break;
                    tc_fence_after();
                    uint32_t a1[32], a2[32];
                    tmem_ld32(tAcc + wg * 32, a1);
                    tmem_ld32(tAcc + 64 + wg * 32, a2);
                    tmem_wait_ld();
                    uint32_t pk[16], dk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int c0 = 2 * i;
                        float l0, l1, d0, d1;
                        if (MODE == MODE_DKV) {
                            const float2 l2 = *reinterpret_cast<const float2 *>(&stats[slot][0][wg * 32 + c0]);
                            const float2 dl = *reinterpret_cast<const float2 *>(&stats[slot][1][wg * 32 + c0]);
                            l0 = l2.x; l1 = l2.y; d0 = dl.x; d1 = dl.y;
                        } else {
                            l0 = l1 = row_l2;
                            d0 = d1 = row_dl;
                        }
                        float p0 = ex2(fmaf(__uint_as_float(a1[c0]), scale_log2, -l0));
                        float p1 = ex2(fmaf(__uint_as_float(a1[c0 + 1]), scale_log2, -l1));
                        if (MODE == MODE_DQ) {
                            // keys beyond the end of the range
                            if (c0 >= valid) p0 = 0.f;
                            if (c0 + 1 >= valid) p1 = 0.f;
                        }
                        const float s0 = p0 * (__uint_as_float(a2[c0]) - d0);
                        const float s1 = p1 * (__uint_as_float(a2[c0 + 1]) - d1);
                        pk[i] = pack_bf16(p0, p1);
                        dk[i] = pack_bf16(s0, s1);
                    }
                    // in place: the bf16 pairs land in the first half of the 32 fp32 columns this
                    // warpgroup has just read, so no other thread's data is touched
                    if (MODE == MODE_DKV) tmem_st16(tAcc + wg * 32, pk);
                    tmem_st16(tAcc + 64 + wg * 32, dk);
                    ++cS[bf];
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(bar(P_READY + bf));
                }
            }
            if (!ok) break;
            g += wi.kv_blocks;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

// delta[bh, r] = sum_d dO[r, d] * O[r, d]: one warp per row, 8 bytes per lane.
__global__ void __launch_bounds__(256)
delta_kernel(const __nv_bfloat16 *__restrict__ dout, const __nv_bfloat16 *__restrict__ out, float *__restrict__ delta,
             int S, int heads, long long stride_b, long long stride_h, long long stride_s, long long n_rows) {
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= n_rows) return;
    const int lane = threadIdx.x & 31;
    const long long bh = row / S;
    const int r = (int)(row % S);
    const long long off = (bh / heads) * stride_b + (bh % heads) * stride_h + (long long)r * stride_s + lane * 4;
    const uint2 a = *reinterpret_cast<const uint2 *>(dout + off);
    const uint2 c = *reinterpret_cast<const uint2 *>(out + off);
    const float2 a0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&a.x));
    const float2 a1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&a.y));
    const float2 c0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&c.x));
    const float2 c1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&c.y));
    float acc = a0.x * c0.x + a0.y * c0.y + a1.x * c1.x + a1.y * c1.y;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) delta[row] = acc;
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
            it.kv_blocks += (seg_len[s] + SUB - 1) / SUB;
            ++it.n_seg;
        }
        items.push_back(it);
    }
}

}  // namespace

// Work list of the backward kernels: 128 resident rows per item, the rows they exchange
// gradients with listed as up to three contiguous ranges and counted in sub-blocks of 64.
// Also allocates the delta scratch.  Called from hilberta_plan_bind for bf16 bindings.
int attn_bwd_prepare(hilberta_plan_t *p) {
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
    cudaFree(p->d_bwd_work);
    cudaFree(p->d_bwd_units);
    cudaFree(p->d_bwd_cta_begin);
    cudaFree(p->d_delta);
    p->d_bwd_work = nullptr;
    p->d_bwd_units = nullptr;
    p->d_bwd_cta_begin = nullptr;
    p->d_delta = nullptr;
    p->n_bwd_work = (int)items.size();
    p->n_bwd_cta = 0;
    if (items.empty()) return HILBERTA_OK;

    const int bh = p->batch * p->heads;
    const long long n_units = (long long)items.size() * bh;
    if (n_units > (1ll << 30)) return HILBERTA_ERR_INVALID;
    const int n_cta = (int)std::min<long long>(n_units, p->sm_count);
    std::vector<std::vector<WorkUnit>> bins(n_cta);
    typedef std::pair<long long, int> Load;
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int c = 0; c < n_cta; ++c) heap.push(Load(0, c));
    for (int i = 0; i < (int)items.size(); ++i) {
        const long long cost = (long long)items[i].kv_blocks + 3;
        for (int j = 0; j < bh; ++j) {
            Load top = heap.top();
            heap.pop();
            bins[top.second].push_back(WorkUnit{i, j});
            heap.push(Load(top.first + cost, top.second));
        }
    }
    std::vector<WorkUnit> units;
    std::vector<int> cta_begin(n_cta + 1, 0);
    units.reserve((size_t)n_units);
    for (int c = 0; c < n_cta; ++c) {
        cta_begin[c] = (int)units.size();
        units.insert(units.end(), bins[c].begin(), bins[c].end());
    }
    cta_begin[n_cta] = (int)units.size();
    p->n_bwd_cta = n_cta;
    HB_CUDA(cudaMalloc(&p->d_bwd_work, sizeof(WorkItem) * items.size()));
    HB_CUDA(cudaMemcpy(p->d_bwd_work, items.data(), sizeof(WorkItem) * items.size(), cudaMemcpyHostToDevice));
    HB_CUDA(cudaMalloc(&p->d_bwd_units, sizeof(WorkUnit) * units.size()));
    HB_CUDA(cudaMemcpy(p->d_bwd_units, units.data(), sizeof(WorkUnit) * units.size(), cudaMemcpyHostToDevice));
    HB_CUDA(cudaMalloc(&p->d_bwd_cta_begin, sizeof(int) * cta_begin.size()));
    HB_CUDA(cudaMemcpy(p->d_bwd_cta_begin, cta_begin.data(), sizeof(int) * cta_begin.size(), cudaMemcpyHostToDevice));
    HB_CUDA(cudaMalloc(&p->d_delta, sizeof(float) * (size_t)bh * p->S));
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(attn_bwd_kernel<MODE_DQ>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes_of(MODE_DQ));
        if (attr_err == cudaSuccess)
            attr_err = cudaFuncSetAttribute(attn_bwd_kernel<MODE_DKV>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            smem_bytes_of(MODE_DKV));
    });
    HB_CUDA(attr_err);
    return HILBERTA_OK;
}

int launch_attn_bwd(const hilberta_plan_t *p, const void *dout, const void *q, const void *k, const void *v,
                    const void *out, const float *lse, void *dq, void *dk, void *dv, float *delta,
                    cudaStream_t stream) {
    if (p->n_bwd_work == 0) return HILBERTA_OK;
    CUtensorMap mq, mk, mv, mdo;
    int rc;
    if ((rc = make_tensor_map(&mq, q, p, SUB)) != HILBERTA_OK) return rc;
    if ((rc = make_tensor_map(&mk, k, p, SUB)) != HILBERTA_OK) return rc;
    if ((rc = make_tensor_map(&mv, v, p, SUB)) != HILBERTA_OK) return rc;
    if ((rc = make_tensor_map(&mdo, dout, p, SUB)) != HILBERTA_OK) return rc;
    const long long n_rows = (long long)p->batch * p->heads * p->S;
    delta_kernel<<<(unsigned)((n_rows + 7) / 8), 256, 0, stream>>>(
        (const __nv_bfloat16 *)dout, (const __nv_bfloat16 *)out, delta, p->S, p->heads, p->stride_b, p->stride_h,
        p->stride_s, n_rows);
    HB_LAUNCHED();
    Params prm;
    prm.work = p->d_bwd_work;
    prm.units = p->d_bwd_units;
    prm.cta_begin = p->d_bwd_cta_begin;
    prm.heads = p->heads;
    prm.stride_b = p->stride_b;
    prm.stride_h = p->stride_h;
    prm.stride_s = p->stride_s;
    prm.lse = lse;
    prm.delta = delta;
    prm.scale = p->scale;
    prm.scale_log2 = p->scale * 1.4426950408889634f;
    prm.S = p->S;
    prm.status = p->d_status;
    prm.out_align32 = ((((uintptr_t)dq | (uintptr_t)dk | (uintptr_t)dv) & 31) == 0 &&
                       ((p->stride_b | p->stride_h | p->stride_s) & 15) == 0) ? 1 : 0;
    prm.out_a = (__nv_bfloat16 *)dq;
    prm.out_b = nullptr;
    attn_bwd_kernel<MODE_DQ><<<p->n_bwd_cta, THREADS, smem_bytes_of(MODE_DQ), stream>>>(mq, mdo, mk, mv, prm);
    HB_LAUNCHED();
    prm.out_a = (__nv_bfloat16 *)dk;
    prm.out_b = (__nv_bfloat16 *)dv;
    attn_bwd_kernel<MODE_DKV><<<p->n_bwd_cta, THREADS, smem_bytes_of(MODE_DKV), stream>>>(mk, mv, mq, mdo, prm);
    HB_LAUNCHED();
    return HILBERTA_OK;
}

}  // namespace hilberta

// ---------------------------------------------------------------------------
// hilberta_backward_static: the same three launches with the delta scratch in a
// fixed array that is part of the library image instead of memory obtained from
// the CUDA allocator.  The array lives on every device that loads the library.
// In host code its name is only a handle; the device address is looked up once
// per device with cudaGetSymbolAddress and cached.
static __device__ __align__(256) float g_static_delta[HILBERTA_STATIC_SCRATCH_FLOATS];

namespace {
constexpr int MAX_DEVICES = 64;
std::mutex g_static_mutex;
float *g_static_delta_ptr[MAX_DEVICES] = {};

// Device address of g_static_delta on `device`, which must be the current device.
int static_delta_address(int device, float **ptr) {
    if (device < 0 || device >= MAX_DEVICES) return HILBERTA_ERR_INVALID;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_delta_ptr[device]) {
        float *addr = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void **)&addr, g_static_delta);
        if (e != cudaSuccess || !addr) {
            hilberta::g_last_cuda_error = (int)e;
            return HILBERTA_ERR_CUDA;
        }
        g_static_delta_ptr[device] = addr;
    }
    *ptr = g_static_delta_ptr[device];
    return HILBERTA_OK;
}
}  // namespace

extern "C" int hilberta_backward_static(const void *dout, const void *q, const void *k, const void *v,
                                        const void *out, const float *lse, void *dq, void *dk, void *dv,
                                        const hilberta_plan_t *p, void *stream) {
    if (!p || !dout || !q || !k || !v || !out || !lse || !dq || !dk || !dv) return HILBERTA_ERR_INVALID;
    if (!p->bound) return HILBERTA_ERR_UNBOUND;
    if (p->dtype != HILBERTA_BF16) return HILBERTA_ERR_UNSUPPORTED;
    const void *in[5] = {dout, q, k, v, out};
    void *outs[3] = {dq, dk, dv};
    uintptr_t bits = ((uintptr_t)lse & 3) ? 15 : 0;
    for (int i = 0; i < 3; ++i) {
        bits |= (uintptr_t)outs[i];
        for (int j = 0; j < 5; ++j)
            if (outs[i] == in[j]) return HILBERTA_ERR_INVALID;
        for (int j = 0; j < i; ++j)
            if (outs[i] == outs[j]) return HILBERTA_ERR_INVALID;
    }
    for (int j = 0; j < 5; ++j) bits |= (uintptr_t)in[j];
    if (bits & 15) return HILBERTA_ERR_INVALID;
    // one float of scratch per (batch, head, token): refuse what the fixed array cannot hold
    if ((unsigned long long)p->batch * p->heads * p->S > (unsigned long long)HILBERTA_STATIC_SCRATCH_FLOATS)
        return HILBERTA_ERR_BUFFER;
    int dev = -1;
    HB_CUDA(cudaGetDevice(&dev));
    if (dev != p->device) return HILBERTA_ERR_INVALID;
    float *delta = nullptr;
    const int rc = static_delta_address(dev, &delta);
    if (rc != HILBERTA_OK) return rc;
    // delta_kernel overwrites every entry the two tensor-core kernels read, so whatever an
    // earlier call left in the array is never seen and nothing has to be cleared
    return hilberta::launch_attn_bwd(p, dout, q, k, v, out, lse, dq, dk, dv, delta, (cudaStream_t)stream);
}
