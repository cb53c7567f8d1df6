// bf16 backward pass of the block-sparse attention for sm_100a.  The paper trains
// through its kernel (Sec. 4.1) without describing the backward pass; this is the
// derivative of Algorithm 1's result on the same physical layout, key lists and
// work items as the forward kernel (the mask is symmetric, so the queries that see
// a key tile are listed exactly like the keys a query tile sees).
//
// With P = exp(s Q K^T - LSE), dP = dO V^T, delta = rowsum(dO * O) and
// dS = P * (dP - delta):   dQ = s dS K,   dK = s dS^T Q,   dV = P^T dO.
//
// Three launches: a bandwidth-bound pass that writes (LSE * log2 e, delta) per row,
// then one tensor-core kernel in two modes that share all code but a few lines.
//   mode DQ : resident tile = 128 query rows (Q_i, dO_i); streamed = their keys (K_j, V_j)
//             A = Q_i K_j^T, B = dO_i V_j^T, dS -> TMEM, dQ_i += dS K_j
//   mode DKV: resident tile = 128 key rows (K_j, V_j); streamed = the queries that see them
//             A = K_j Q_i^T, B = V_j dO_i^T (transposed scores: a thread owns a KEY row),
//             P^T, dS^T -> TMEM, dV_j += P^T dO_i, dK_j += dS^T Q_i
// Streamed rows come in blocks of 128.  TMEM: region A (scores, 128 columns), region B (dP,
// 128 columns), outputs.  The element-wise step works in two phases: phase 1 turns the scores
// into weights as soon as A is written and releases A at once, so the scores of the NEXT block
// are computed while phase 2 (which needs B) and the output MMAs of this block run; phase 2
// overwrites B in place with P and dS (bf16), each thread inside the 32 columns it has just
// read.  Per block the tensor pipe sees  A(s+1) | out(s) | B(s+1)  back to back.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <functional>
#include <mutex>
#include <queue>
#include <type_traits>
#include <utility>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace hilberta {
using namespace ptx;

int make_tensor_map(CUtensorMap *m, const void *base, const hilberta_plan_t *p, int box_rows, int heads = 0);

namespace {

constexpr int BM = 128;   // resident rows per work item
constexpr int BK = 128;   // streamed rows per block
constexpr int TILE_BYTES = BM * 128 * 2;  // 32 KB slot: two 64-column slabs of 128 rows (head dim 64 uses the first)
constexpr int SLAB_BYTES = TILE_BYTES / 2;
constexpr int NT1 = 3;    // ring of the streamed operand that is read twice (scores early, output MMA late)
constexpr int NT2 = 2;    // ring of the streamed operand of dP
constexpr int STAT_BYTES = 2 * BK * 4;      // lse2[128] then delta[128] of a block's streamed rows (DKV)
constexpr int THREADS = 512;  // 8 element-wise warps, 4 single-lane service warps, 4 epilogue warps
constexpr uint32_t TMEM_COLS = 512;
constexpr int MODE_DQ = 0, MODE_DKV = 1;

enum Bar {
    RES_FULL = 0, RES_EMPTY, OUT_FULL, EPI_DONE, DRAIN,
    S_FULL,       // region A written
    A_DONE,       // region A read by every element-wise thread (256 arrivals)
    DP_FULL,      // region B written
    P_READY,      // P / dS written over region B (256 arrivals)
    T1_FULL, T1_EMPTY = T1_FULL + NT1,
    T2_FULL = T1_EMPTY + NT1, T2_EMPTY = T2_FULL + NT2,
    NUM_BARS = T2_EMPTY + NT2
};

// shared memory map (all dynamic; the tile area must start on a 1024-byte boundary)
constexpr int OFF_R1 = 0, OFF_R2 = TILE_BYTES, OFF_T1 = 2 * TILE_BYTES, OFF_T2 = OFF_T1 + NT1 * TILE_BYTES;
constexpr int OFF_STAT = OFF_T2 + NT2 * TILE_BYTES;
constexpr int OFF_BARS = OFF_STAT + NT2 * STAT_BYTES;
constexpr int OFF_MISC = OFF_BARS + NUM_BARS * 8;
constexpr int SMEM_USED = OFF_MISC + 16;
constexpr int SMEM_BYTES = 232448;   // the 227 KB a CTA may have; SMEM_USED plus the alignment gap must fit

struct Params {
    const WorkItem *work;
    const WorkUnit *units;
    const int *cta_begin;
    int heads;
    long long stride_b, stride_h, stride_s;  // elements
    const float *lse2;    // [batch * heads * S] lse * log2 e
    const float *delta;   // [batch * heads * S] rowsum(dO * O)
    __nv_bfloat16 *out_a; // DQ: dq; DKV: dk
    __nv_bfloat16 *out_b; // DKV: dv
    float scale, scale_log2;
    int S;
    int out_align32;      // outputs and strides 32-byte aligned: 32-byte stores allowed
    int *status;
};

__device__ __forceinline__ int seg_blocks(const WorkItem &it, int seg) {
    return (it.seg_len[seg] + BK - 1) / BK;
}

__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}

// acc = R T^T: resident tile (128 rows) times a streamed block (128 rows), K = head dim.
template <int HD>
__device__ __forceinline__ void issue_rt(uint32_t tmem_acc, uint32_t sR, uint32_t sT) {
    constexpr uint32_t IDESC = idesc_bf16_f32(BM, BK, 0, 0);
    const uint64_t da = smem_desc_sw128(sR, 16, 1024), db = smem_desc_sw128(sT, 16, 1024);
#pragma unroll
    for (int k = 0; k < HD / 16; ++k) {
        const uint64_t off = (uint64_t)(((k >> 2) * SLAB_BYTES + (k & 3) * 32) >> 4);
        mma_ss(tmem_acc, da + off, db + off, IDESC, k > 0);
    }
}

// out (+)= A T: A (128 x 128, bf16) from TMEM, the streamed block row-major in smem (N-major
// operand: 128 rows of K, two 64-column slabs of N).  The bf16 pairs of streamed rows
// [32 g, 32 g + 32) sit 16 columns wide at column 32 g of region B (+ a_off).
template <int HD>
__device__ __forceinline__ void issue_at(uint32_t tmem_out, uint32_t tmem_b, uint32_t a_off, uint32_t sT,
                                         bool accumulate) {
    constexpr uint32_t IDESC = idesc_bf16_f32(BM, HD, 0, 1);
    const uint64_t db = smem_desc_sw128(sT, SLAB_BYTES, 1024);
#pragma unroll
    for (int k = 0; k < BK / 16; ++k)
        mma_ts(tmem_out, tmem_b + (k >> 1) * 32 + a_off + (k & 1) * 8, db + (uint64_t)((k * 2048) >> 4), IDESC,
               (accumulate || k > 0) ? 1u : 0u);
}

template <int MODE, int HD>
__global__ void __launch_bounds__(THREADS, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmR1, const __grid_constant__ CUtensorMap tmR2,
                const __grid_constant__ CUtensorMap tmT1, const __grid_constant__ CUtensorMap tmT2,
                const Params prm) {
    extern __shared__ uint8_t smem_raw[];
#ifdef HB_STAMPS
    if (threadIdx.x == 0) {
        unsigned long long ns;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
        prm.status[1024 + MODE * 1024 + 4 * blockIdx.x] = (int)(ns & 0x7fffffff);
    }
#endif
    constexpr uint32_t REG_A = 0, REG_B = 128, OUT_A = 256, OUT_B = 384;   // TMEM columns
    constexpr int NSLAB = HD / 64;
    constexpr uint32_t TILE_TX = BM * HD * 2;                              // bytes of one tile

    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    if ((int)(smem - smem_raw) + SMEM_USED > SMEM_BYTES) {
        // the dynamic area starts too far from a 1024-byte boundary for everything to fit
        if (threadIdx.x == 0 && atomicCAS(prm.status, 0, 0x900) == 0) prm.status[1] = blockIdx.x;
        return;
    }
    const uint32_t sbase = smem_u32(smem);
    const uint32_t sR1 = sbase + OFF_R1, sR2 = sbase + OFF_R2, sT1 = sbase + OFF_T1, sT2 = sbase + OFF_T2;
    const float *stats = reinterpret_cast<const float *>(smem + OFF_STAT);
    const uint32_t bar0 = sbase + OFF_BARS;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + OFF_MISC);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + OFF_MISC + 4);
    const int tid = threadIdx.x, warp = tid >> 5;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        *abort_flag = 0;
        for (int i = 0; i < NUM_BARS; ++i) {
            uint32_t count = 1;
            if (i == EPI_DONE) count = 128;
            if (i == A_DONE || i == P_READY) count = 256;
            // DKV: ring 2 also carries the row statistics, copied by the 32 lanes of its producer warp
            if (MODE == MODE_DKV && i >= T2_FULL && i < T2_FULL + NT2) count = 33;
            mbar_init(bar(i), count);
        }
        mbar_fence_init();
    }
    if (warp == 8) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int u_begin = prm.cta_begin[blockIdx.x], u_end = prm.cta_begin[blockIdx.x + 1];

    if (warp >= 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
    }
    if (warp == 8 || warp == 10) {
        // ------------------------------------------------ producers of the streamed blocks
        // warp 8 feeds ring 1 (K_j in DQ mode, Q_i in DKV mode), warp 10 ring 2 (V_j / dO_i and,
        // in DKV mode, the statistics of the streamed query rows)
        const bool second = warp == 10;
        const int lane = tid & 31;
        const bool with_stats = MODE == MODE_DKV && second;   // whole warp takes part
        const bool leader = with_stats ? lane == 0 : elect_one();
        if (leader || with_stats) {
            const CUtensorMap *tm = second ? &tmT2 : &tmT1;
            if (leader) prefetch_tmap(tm);
            const int nslot = second ? NT2 : NT1;
            const int FULL = second ? T2_FULL : T1_FULL, EMPTY = second ? T2_EMPTY : T1_EMPTY;
            const uint32_t ring = second ? sT2 : sT1;
            uint32_t g = 0;
            bool ok = true;
            for (int u = u_begin; ok && u < u_end; ++u) {
                const WorkUnit unit = prm.units[u];
                const WorkItem wi = prm.work[unit.item];
                const int b = unit.bh / prm.heads, h = unit.bh % prm.heads;
                for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                    const int nb = seg_blocks(wi, seg);
                    for (int j = 0; j < nb; ++j, ++g) {
                        const int row = wi.seg_start[seg] + j * BK;
                        const uint32_t s = g % nslot, ph = (g / nslot) & 1;
                        if (leader) ok = wait_or_abort(bar(EMPTY + s), ph ^ 1, abort_flag, prm.status, 0x402 + (second ? 1 : 0));
                        if (with_stats) ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                        if (!ok) break;
                        if (leader) {
                            const uint32_t dst = ring + s * TILE_BYTES;
                            mbar_expect_tx(bar(FULL + s), TILE_TX);
#pragma unroll
                            for (int sl = 0; sl < NSLAB; ++sl)
                                tma_load_4d(dst + sl * SLAB_BYTES, tm, bar(FULL + s), 64 * sl, row, h, b);
                        }
                        if (with_stats) {
                            // lse2 and delta of the block's rows that lie inside the range (the others
                            // are masked by position later); the arrival fires when the copies land
                            const int valid = min(BK, wi.seg_len[seg] - j * BK);
                            const long long p0 = (long long)unit.bh * prm.S + row;
                            const uint32_t sdst = sbase + OFF_STAT + s * STAT_BYTES;
#pragma unroll
                            for (int i = 0; i < BK / 32; ++i) {
                                const int c = lane + 32 * i;
                                if (c < valid) {
                                    cp_async4(sdst + 4 * c, prm.lse2 + p0 + c);
                                    cp_async4(sdst + 4 * (BK + c), prm.delta + p0 + c);
                                }
                            }
                            asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar(FULL + s)) : "memory");
                        }
                    }
                }
            }
            if (with_stats) asm volatile("cp.async.wait_all;" ::: "memory");
            if (!ok && leader) {
                // let every copy already issued land before the CTA retires
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000) {
                }
            }
        }
    } else if (warp == 11) {
        // ------------------------------------------------ loader of the resident tiles
        // A thread of its own, so that the block producers can run ahead into the next unit
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
                if (uc > 0) ok = wait_or_abort(bar(RES_EMPTY), (uc - 1) & 1, abort_flag, prm.status, 0x401);
                if (!ok) break;
                mbar_expect_tx(bar(RES_FULL), 2 * TILE_TX);
#pragma unroll
                for (int sl = 0; sl < NSLAB; ++sl) {
                    tma_load_4d(sR1 + sl * SLAB_BYTES, &tmR1, bar(RES_FULL), 64 * sl, wi.q_start, h, b);
                    tma_load_4d(sR2 + sl * SLAB_BYTES, &tmR2, bar(RES_FULL), 64 * sl, wi.q_start, h, b);
                }
                if (u + 1 < u_end) {
                    // pull the next unit's resident tiles into L2 while this unit runs
                    const WorkUnit nu = prm.units[u + 1];
                    const int nq = prm.work[nu.item].q_start;
                    const int nb_ = nu.bh / prm.heads, nh = nu.bh % prm.heads;
#pragma unroll
                    for (int sl = 0; sl < NSLAB; ++sl) {
                        tma_prefetch_4d(&tmR1, 64 * sl, nq, nh, nb_);
                        tma_prefetch_4d(&tmR2, 64 * sl, nq, nh, nb_);
                    }
                }
            }
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000) {
                }
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
            ok = wait_or_abort(bar(OUT_FULL), uc & 1, abort_flag, prm.status, 0x605);
            if (!ok) break;
            tc_fence_after();
            const long long roff = (long long)b * prm.stride_b + (long long)h * prm.stride_h +
                                   (long long)(wi.q_start + r) * prm.stride_s;
            constexpr int CPO = HD / 32;                              // 32-column chunks per output
            constexpr int NCH = (MODE == MODE_DKV) ? 2 * CPO : CPO;   // DKV: dK then dV
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                uint32_t o[32];
                tmem_ld32(tmem + lane_addr + (c >= CPO ? OUT_B + (c - CPO) * 32 : OUT_A + c * 32), o);
                tmem_wait_ld();
                if (row_ok) {
                    __nv_bfloat16 *orow = (c >= CPO ? prm.out_b : prm.out_a) + roff + (c % CPO) * 32;
                    const float mul = c >= CPO ? 1.f : prm.scale;
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
            uint32_t g = 0, uc = 0;   // g: blocks issued so far (ring positions and barrier phases)
            bool ok = true;
            auto t1 = [&](uint32_t e) { return sT1 + (e % NT1) * TILE_BYTES; };
            auto t2 = [&](uint32_t e) { return sT2 + (e % NT2) * TILE_BYTES; };
            for (int u = u_begin; ok && u < u_end; ++u, ++uc) {
                const WorkItem wi = prm.work[prm.units[u].item];
                const int n = wi.kv_blocks;  // blocks of this item
                ok = wait_or_abort(bar(RES_FULL), uc & 1, abort_flag, prm.status, 0x501);
                if (!ok) break;
                // scores and dP of the first block
                ok = wait_or_abort(bar(T1_FULL + g % NT1), (g / NT1) & 1, abort_flag, prm.status, 0x502);
                if (!ok) break;
                tc_fence_after();
                issue_rt<HD>(tmem + REG_A, sR1, t1(g));
                mma_commit(bar(S_FULL));
                ok = wait_or_abort(bar(T2_FULL + g % NT2), (g / NT2) & 1, abort_flag, prm.status, 0x503);
                if (!ok) break;
                tc_fence_after();
                issue_rt<HD>(tmem + REG_B, sR2, t2(g));
                mma_commit(bar(DP_FULL));
                if (MODE == MODE_DQ) mma_commit(bar(T2_EMPTY + g % NT2));
                if (n == 1) mma_commit(bar(RES_EMPTY));
                for (int s = 0; s < n; ++s) {
                    const uint32_t e = g + s;
                    const bool more = s + 1 < n;
                    if (more) {
                        // scores of the next block, as soon as phase 1 has read this block's
                        ok = wait_or_abort(bar(T1_FULL + (e + 1) % NT1), ((e + 1) / NT1) & 1, abort_flag, prm.status, 0x504);
                        if (!ok) break;
                        ok = wait_or_abort(bar(A_DONE), e & 1, abort_flag, prm.status, 0x505);
                        if (!ok) break;
                        tc_fence_after();
                        issue_rt<HD>(tmem + REG_A, sR1, t1(e + 1));
                        mma_commit(bar(S_FULL));
                    }
                    if (s == 0 && uc > 0) {
                        // the previous unit's accumulators have been read out
                        ok = wait_or_abort(bar(EPI_DONE), (uc - 1) & 1, abort_flag, prm.status, 0x506);
                        if (!ok) break;
                    }
                    ok = wait_or_abort(bar(P_READY), e & 1, abort_flag, prm.status, 0x507);
                    if (!ok) break;
                    tc_fence_after();
                    issue_at<HD>(tmem + OUT_A, tmem + REG_B, 16, t1(e), s > 0);                       // dS  x T1
                    if (MODE == MODE_DKV) issue_at<HD>(tmem + OUT_B, tmem + REG_B, 0, t2(e), s > 0);   // P^T x T2
                    mma_commit(bar(T1_EMPTY + e % NT1));
                    if (MODE == MODE_DKV) mma_commit(bar(T2_EMPTY + e % NT2));
                    if (more) {
                        // dP of the next block overwrites P / dS of this one: after the MMAs above
                        ok = wait_or_abort(bar(T2_FULL + (e + 1) % NT2), ((e + 1) / NT2) & 1, abort_flag, prm.status, 0x508);
                        if (!ok) break;
                        tc_fence_after();
                        issue_rt<HD>(tmem + REG_B, sR2, t2(e + 1));
                        mma_commit(bar(DP_FULL));
                        if (MODE == MODE_DQ) mma_commit(bar(T2_EMPTY + (e + 1) % NT2));
                        if (s + 2 == n) mma_commit(bar(RES_EMPTY));   // last read of the resident tiles
                    }
                }
                if (!ok) break;
                mma_commit(bar(OUT_FULL));
                g += n;
            }
            // every MMA issued above has retired before TMEM is released
            mma_commit(bar(DRAIN));
            wait_or_abort(bar(DRAIN), 0, abort_flag, prm.status, 0x509);
        }
    } else if (warp < 8) {
        // ------------------------------------ element-wise step, warpgroup wg: columns [64 wg, +64)
        asm volatile("setmaxnreg.inc.sync.aligned.u32 168;");
        const int wg = warp >> 2;
        const int r = tid & 127;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tA = tmem + lane_addr + REG_A + wg * 64, tB = tmem + lane_addr + REG_B + wg * 64;
        const float scale_log2 = prm.scale_log2;
        uint32_t g = 0;
        bool ok = true;
        for (int u = u_begin; ok && u < u_end; ++u) {
            const WorkUnit unit = prm.units[u];
            const WorkItem wi = prm.work[unit.item];
            const int bh = unit.bh;
            // DQ: this thread's query row statistics; rows beyond the item get lse = +inf,
            // which turns their weights into exact zeros
            float row_l2 = __int_as_float(0x7f800000), row_dl = 0.f;
            if (MODE == MODE_DQ && r < wi.q_rows) {
                row_l2 = __ldg(prm.lse2 + (long long)bh * prm.S + wi.q_start + r);
                row_dl = __ldg(prm.delta + (long long)bh * prm.S + wi.q_start + r);
            }
            for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                const int nb = seg_blocks(wi, seg);
                for (int j = 0; j < nb; ++j, ++g) {
                    // streamed rows of this warpgroup that lie inside the range
                    const int valid = min(BK, wi.seg_len[seg] - j * BK) - wg * 64;
                    const float4 *st_l = nullptr, *st_d = nullptr;
                    if (MODE == MODE_DKV) {
                        // the statistics arrive with ring 2
                        ok = wait_or_abort(bar(T2_FULL + g % NT2), (g / NT2) & 1, abort_flag, prm.status, 0x601 + wg);
                        if (!ok) break;
                        st_l = reinterpret_cast<const float4 *>(stats + (g % NT2) * (2 * BK) + wg * 64);
                        st_d = st_l + BK / 4;
                    }
                    // ---- phase 1: weights from the scores
                    ok = wait_or_abort(bar(S_FULL), g & 1, abort_flag, prm.status, 0x603 + wg);
                    if (!ok) break;
                    tc_fence_after();
                    uint32_t a[64];
                    tmem_ld32(tA, *reinterpret_cast<uint32_t(*)[32]>(&a[0]));
                    tmem_ld32(tA + 32, *reinterpret_cast<uint32_t(*)[32]>(&a[32]));
                    tmem_wait_ld();
                    tc_fence_before();
                    mbar_arrive(bar(A_DONE));   // region A may take the next block's scores
                    const bool ragged = valid < 64;   // only the last block of a range
                    auto phase1 = [&](auto RAGGED) {
#pragma unroll
                        for (int c4 = 0; c4 < 16; ++c4) {
                            float4 l4 = make_float4(row_l2, row_l2, row_l2, row_l2);
                            if (MODE == MODE_DKV) l4 = st_l[c4];
                            const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(a[4 * c4]), __uint_as_float(a[4 * c4 + 1])),
                                                         make_float2(scale_log2, scale_log2), make_float2(-l4.x, -l4.y));
                            const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(a[4 * c4 + 2]), __uint_as_float(a[4 * c4 + 3])),
                                                         make_float2(scale_log2, scale_log2), make_float2(-l4.z, -l4.w));
                            // (a polynomial exp2 on the FMA pipes for part of the pairs, as in the forward
                            // kernel, measured equal here: this step is not bound by the MUFU unit)
                            float2 p0, p1;
                            p0.x = ex2(x0.x);
                            p0.y = ex2(x0.y);
                            p1.x = ex2(x1.x);
                            p1.y = ex2(x1.y);
                            if (decltype(RAGGED)::value) {
                                // rows beyond the end of the range (their statistics are stale)
                                if (4 * c4 >= valid) p0.x = 0.f;
                                if (4 * c4 + 1 >= valid) p0.y = 0.f;
                                if (4 * c4 + 2 >= valid) p1.x = 0.f;
                                if (4 * c4 + 3 >= valid) p1.y = 0.f;
                            }
                            a[4 * c4] = __float_as_uint(p0.x);
                            a[4 * c4 + 1] = __float_as_uint(p0.y);
                            a[4 * c4 + 2] = __float_as_uint(p1.x);
                            a[4 * c4 + 3] = __float_as_uint(p1.y);
                        }
                    };
                    if (ragged) phase1(std::true_type{});
                    else phase1(std::false_type{});
                    // ---- phase 2: dS = P * (dP - delta), written over dP together with P
                    ok = wait_or_abort(bar(DP_FULL), g & 1, abort_flag, prm.status, 0x605 + wg);
                    if (!ok) break;
                    tc_fence_after();
                    auto phase2 = [&](auto RAGGED) {
#pragma unroll
                        for (int h2 = 0; h2 < 2; ++h2) {
                            uint32_t d[32];
                            tmem_ld32(tB + h2 * 32, d);
                            tmem_wait_ld();
                            uint32_t pk[16], dk[16];
#pragma unroll
                            for (int i4 = 0; i4 < 8; ++i4) {
                                const int c0 = h2 * 32 + 4 * i4;
                                float4 d4 = make_float4(row_dl, row_dl, row_dl, row_dl);
                                if (MODE == MODE_DKV) d4 = st_d[c0 >> 2];
                                const float2 pa = make_float2(__uint_as_float(a[c0]), __uint_as_float(a[c0 + 1]));
                                const float2 pb = make_float2(__uint_as_float(a[c0 + 2]), __uint_as_float(a[c0 + 3]));
                                float2 sa = __fadd2_rn(make_float2(__uint_as_float(d[4 * i4]), __uint_as_float(d[4 * i4 + 1])),
                                                       make_float2(-d4.x, -d4.y));
                                float2 sb = __fadd2_rn(make_float2(__uint_as_float(d[4 * i4 + 2]), __uint_as_float(d[4 * i4 + 3])),
                                                       make_float2(-d4.z, -d4.w));
                                sa = __fmul2_rn(sa, pa);
                                sb = __fmul2_rn(sb, pb);
                                if (decltype(RAGGED)::value) {
                                    // P is zero there already; dP - delta may be anything
                                    if (c0 >= valid) sa.x = 0.f;
                                    if (c0 + 1 >= valid) sa.y = 0.f;
                                    if (c0 + 2 >= valid) sb.x = 0.f;
                                    if (c0 + 3 >= valid) sb.y = 0.f;
                                }
                                pk[2 * i4] = pack_bf16(pa.x, pa.y);
                                pk[2 * i4 + 1] = pack_bf16(pb.x, pb.y);
                                dk[2 * i4] = pack_bf16(sa.x, sa.y);
                                dk[2 * i4 + 1] = pack_bf16(sb.x, sb.y);
                            }
                            // the 32 columns just read take P (16 columns of bf16 pairs) and dS (16)
                            if (MODE == MODE_DKV) tmem_st16(tB + h2 * 32, pk);
                            tmem_st16(tB + h2 * 32 + 16, dk);
                        }
                    };
                    if (ragged) phase2(std::true_type{});
                    else phase2(std::false_type{});
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(bar(P_READY));
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tmem_dealloc(tmem, TMEM_COLS);
    }
#ifdef HB_STAMPS
    if (threadIdx.x == 0) {
        unsigned long long ns;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
        prm.status[1024 + MODE * 1024 + 4 * blockIdx.x + 1] = (int)(ns & 0x7fffffff);
    }
#endif
}

// lse2[row] = lse[row] * log2 e, delta[row] = sum_d dO[row, d] * O[row, d]: HD / 8 lanes per row
// (16 bytes each), four rows in flight per lane group.
template <int HD>
__global__ void __launch_bounds__(256)
delta_kernel(const __nv_bfloat16 *__restrict__ dout, const __nv_bfloat16 *__restrict__ out,
             const float *__restrict__ lse, float *__restrict__ lse2, float *__restrict__ delta, int S, int heads,
             long long stride_b, long long stride_h, long long stride_s, long long n_rows) {
    constexpr int LPR = HD / 8;   // lanes per row (16 bytes each)
    const int sub = threadIdx.x % LPR;
    const long long row0 = ((long long)blockIdx.x * (256 / LPR) + threadIdx.x / LPR) * 4;
    uint4 a[4], c[4];
    bool in[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const long long row = row0 + i;
        in[i] = row < n_rows;
        if (in[i]) {
            const long long bh = row / S;
            const long long off = (bh / heads) * stride_b + (bh % heads) * stride_h + (row % S) * stride_s + sub * 8;
            a[i] = *reinterpret_cast<const uint4 *>(dout + off);
            c[i] = *reinterpret_cast<const uint4 *>(out + off);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float acc = 0.f;
        if (in[i]) {
            const uint32_t *ua = reinterpret_cast<const uint32_t *>(&a[i]), *uc = reinterpret_cast<const uint32_t *>(&c[i]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ua[e]));
                const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&uc[e]));
                acc = fmaf(x.x, y.x, fmaf(x.y, y.y, acc));
            }
        }
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (in[i] && sub == 0) {
            lse2[row0 + i] = lse[row0 + i] * 1.4426950408889634f;
            delta[row0 + i] = acc;
        }
    }
}

}  // namespace

// Work list of the backward kernels: 128 resident rows per item, the rows they exchange
// gradients with listed as up to three contiguous ranges and counted in blocks of 128.
// Also allocates the per-row scratch: lse * log2 e for every row, then delta for every row.  Called from hilberta_plan_bind for bf16 bindings.
int attn_bwd_prepare(hilberta_plan_t *p) {
    std::vector<WorkItem> items = build_work_items(p, BM, BK);
    {
        const int rc_items = check_work_items(items.data(), (int)items.size(), p->S, BM, BK);
        if (rc_items != HILBERTA_OK) return rc_items;
    }
    std::stable_sort(items.begin(), items.end(),
                     [](const WorkItem &a, const WorkItem &b) { return a.kv_blocks > b.kv_blocks; });
    std::vector<long long> cost;
    for (const WorkItem &it : items) cost.push_back((long long)it.kv_blocks + 3);
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
    HB_CUDA(cudaMalloc(&p->d_bwd_work, sizeof(WorkItem) * items.size()));
    HB_CUDA(cudaMemcpy(p->d_bwd_work, items.data(), sizeof(WorkItem) * items.size(), cudaMemcpyHostToDevice));
    const int rc = upload_schedule(items, cost, bh, p->sm_count, &p->d_bwd_units, &p->d_bwd_cta_begin, &p->n_bwd_cta);
    if (rc != HILBERTA_OK) return rc;
    HB_CUDA(cudaMalloc(&p->d_delta, sizeof(float) * 2 * (size_t)bh * p->S));
    {
        // The shared-memory opt-in is an attribute of the kernel ON ONE DEVICE: set it once for every
        // device a plan is bound on (a failure is reported, not remembered).
        static std::mutex attr_mutex;
        static bool attr_done[64] = {};
        std::lock_guard<std::mutex> lock(attr_mutex);
        if (p->device < 0 || p->device >= 64) return HILBERTA_ERR_INVALID;
        if (!attr_done[p->device]) {
            const void *kernels[4] = {(const void *)attn_bwd_kernel<MODE_DQ, 128>, (const void *)attn_bwd_kernel<MODE_DKV, 128>,
                                      (const void *)attn_bwd_kernel<MODE_DQ, 64>, (const void *)attn_bwd_kernel<MODE_DKV, 64>};
            for (int i = 0; i < 4; ++i)
                HB_CUDA(cudaFuncSetAttribute(kernels[i], cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
            attr_done[p->device] = true;
        }
    }
    return HILBERTA_OK;
}

int launch_attn_bwd(const hilberta_plan_t *p, const void *dout, const void *q, const void *k, const void *v,
                    const void *out, const float *lse, void *dq, void *dk, void *dv, float *delta,
                    cudaStream_t stream) {
    if (p->dtype == HILBERTA_FP8_E4M3) return HILBERTA_ERR_UNSUPPORTED;  // e4m3 bindings are forward only
    if (p->dtype == HILBERTA_FP32)
        return launch_attn_fp32_bwd(p, dout, q, k, v, out, lse, dq, dk, dv, delta, stream);
    if (p->n_bwd_work == 0) return HILBERTA_OK;
    CUtensorMap mq, mk, mv, mdo;
    int rc;
    if ((rc = make_tensor_map(&mq, q, p, BK)) != HILBERTA_OK) return rc;
    if ((rc = make_tensor_map(&mk, k, p, BK)) != HILBERTA_OK) return rc;
    if ((rc = make_tensor_map(&mv, v, p, BK)) != HILBERTA_OK) return rc;
    if ((rc = make_tensor_map(&mdo, dout, p, BK)) != HILBERTA_OK) return rc;
    const long long n_rows = (long long)p->batch * p->heads * p->S;
    if (p->head_dim == 128)
        delta_kernel<128><<<(unsigned)((n_rows + 63) / 64), 256, 0, stream>>>(
            (const __nv_bfloat16 *)dout, (const __nv_bfloat16 *)out, lse, delta, delta + n_rows, p->S, p->heads,
            p->stride_b, p->stride_h, p->stride_s, n_rows);
    else
        delta_kernel<64><<<(unsigned)((n_rows + 127) / 128), 256, 0, stream>>>(
            (const __nv_bfloat16 *)dout, (const __nv_bfloat16 *)out, lse, delta, delta + n_rows, p->S, p->heads,
            p->stride_b, p->stride_h, p->stride_s, n_rows);
    HB_LAUNCHED();
    Params prm;
    prm.work = p->d_bwd_work;
    prm.units = p->d_bwd_units;
    prm.cta_begin = p->d_bwd_cta_begin;
    prm.heads = p->heads;
    prm.stride_b = p->stride_b;
    prm.stride_h = p->stride_h;
    prm.stride_s = p->stride_s;
    prm.lse2 = delta;
    prm.delta = delta + n_rows;
    prm.scale = p->scale;
    prm.scale_log2 = p->scale * 1.4426950408889634f;
    prm.S = p->S;
    prm.status = p->d_status;
    prm.out_align32 = ((((uintptr_t)dq | (uintptr_t)dk | (uintptr_t)dv) & 31) == 0 &&
                       ((p->stride_b | p->stride_h | p->stride_s) & 15) == 0) ? 1 : 0;
    prm.out_a = (__nv_bfloat16 *)dq;
    prm.out_b = nullptr;
    if (p->head_dim == 128)
        attn_bwd_kernel<MODE_DQ, 128><<<p->n_bwd_cta, THREADS, SMEM_BYTES, stream>>>(mq, mdo, mk, mv, prm);
    else
        attn_bwd_kernel<MODE_DQ, 64><<<p->n_bwd_cta, THREADS, SMEM_BYTES, stream>>>(mq, mdo, mk, mv, prm);
    HB_LAUNCHED();
    prm.out_a = (__nv_bfloat16 *)dk;
    prm.out_b = (__nv_bfloat16 *)dv;
    if (p->head_dim == 128)
        attn_bwd_kernel<MODE_DKV, 128><<<p->n_bwd_cta, THREADS, SMEM_BYTES, stream>>>(mk, mv, mq, mdo, prm);
    else
        attn_bwd_kernel<MODE_DKV, 64><<<p->n_bwd_cta, THREADS, SMEM_BYTES, stream>>>(mk, mv, mq, mdo, prm);
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
    // two floats of scratch per (batch, head, token): refuse what the fixed array cannot hold
    if (2ull * p->batch * p->heads * p->S > (unsigned long long)HILBERTA_STATIC_SCRATCH_FLOATS)
        return HILBERTA_ERR_BUFFER;
    const void *in[5] = {dout, q, k, v, out};
    void *outs[3] = {dq, dk, dv};
    uintptr_t bits = ((uintptr_t)lse & 3) ? 15 : 0;
    const size_t esz = p->dtype == HILBERTA_FP32 ? 4 : 2;
    for (int i = 0; i < 3; ++i) {
        bits |= (uintptr_t)outs[i];
        for (int j = 0; j < 5; ++j)
            if (hilberta::bound_tensors_overlap(p, outs[i], esz, in[j], esz)) return HILBERTA_ERR_INVALID;
        for (int j = 0; j < i; ++j)
            if (hilberta::bound_tensors_overlap(p, outs[i], esz, outs[j], esz)) return HILBERTA_ERR_INVALID;
    }
    for (int j = 0; j < 5; ++j) bits |= (uintptr_t)in[j];
    if (bits & 15) return HILBERTA_ERR_INVALID;
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
