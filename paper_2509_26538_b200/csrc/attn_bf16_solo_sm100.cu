// bf16 block-sparse flash-attention forward for sm_100a with ONE query tile per CTA and the scores
// double-buffered (Algorithm 1, restated for Blackwell): head dim 128, inputs in physical order.
//
// A work item is up to 128 consecutive physical query rows that share a key list of up to three
// contiguous ranges, cut into blocks of 128 keys.  With a single query tile per SM, tensor memory
// has room for two score buffers next to the weights and the accumulator:
//
//   TMEM columns:  S_0 [0,128)  S_1 [128,256)  P_0 [256,320)  P_1 [320,384)  O [384,512)
//
// Key block G (counted over the whole launch) uses buffer G & 1 and is handled by softmax
// warpgroup G & 1: it reads S_(G&1) into registers and releases the buffer at once, so Q K^T of
// block G + 2 runs while block G's exponentials are computed, and P V of block G runs while the
// other warpgroup works on block G + 1.  Neither MMA sits on the softmax's dependency chain.
// The two warpgroups own the same rows: they keep separate row sums and share the rows' reference
// maximum through shared memory.  The price is K/V traffic: every K and V tile serves 128 query
// rows instead of 256.
//
// The MMA issuer and the producer treat all key blocks of all the CTA's work items as ONE stream
// (Q K^T runs two blocks ahead of P V, across item boundaries; query tiles are double-buffered).
// Roles inside a CTA (384 threads): warps 0-3 / 4-7 softmax warpgroups 0 / 1 (thread r of a group
// owns row r = TMEM lane r), warp 8 TMA producer, warp 9 MMA issuer, warps 10-11 register donors.
// Every wait is bounded.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <mutex>

#include "attn_softmax_math.cuh"
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace hilberta {
using namespace ptx;

namespace {

constexpr int BM = 128;           // query rows per CTA
constexpr int BN = 128;           // keys per block
constexpr int HD = 128;           // head dim
constexpr int ITEM_ROWS = BM;     // rows per work item
constexpr int Q_BYTES = BM * HD * 2;          // one CTA's query tile: two 64-column slabs
constexpr int TILE_BYTES = BN * HD * 2;       // a K or V tile: 32 KB, two 64-column slabs of 128 rows
constexpr int NSLOT = 4;                      // ring of K / V tiles
constexpr int THREADS = 384;
constexpr int SMEM_BYTES = 2 * Q_BYTES + NSLOT * TILE_BYTES + 1024;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t COL_S = 0, COL_P = 256, COL_O = 384;
constexpr float RESCALE_THRESHOLD = 8.0f;     // log2 units

enum Bar {
    Q_FULL = 0,                    // [2]  the query tile has landed (byte count)
    Q_EMPTY = Q_FULL + 2,          // [2]  each CTA: the unit's last Q K^T has read the tile
    KV_FULL = Q_EMPTY + 2,         // [NSLOT] the tile has landed
    KV_EMPTY = KV_FULL + NSLOT,    // [NSLOT] each CTA: the MMAs reading the slot are done
    S_FULL = KV_EMPTY + NSLOT,     // [2]  each CTA: scores of a block are in S_b
    S_FREE = S_FULL + 2,           // [2]  the group's warps have read S_b (4 arrivals)
    P_READY = S_FREE + 2,          // [2][2] keys [64 h, +64) of P_b written (4 arrivals)
    PV_DONE = P_READY + 4,         // [4]  each CTA: P V of block G done, barrier G & 3
    O_FREE = PV_DONE + 4,          // the epilogue has read O (4 arrivals)
    PUB = O_FREE + 1,              // [2][4] this CTA: warp q of group w published its rows' maximum (one arrival per warp)
    POST = PUB + 8,                // [2][4] this CTA: warp q of group w posted its row sums for an item it does not finish
    ACK = POST + 8,                // [2][4] this CTA: the other group has read that post
    CONS = ACK + 8,                // [2][4] this CTA: the other group has consumed group w's last publication of an item
    DRAIN = CONS + 8,
    NUM_BARS
};

struct SoloParams {
    const WorkItem *work;
    const WorkUnit *units;   // (item, batch*heads index), grouped by CTA
    const int *cta_begin;    // [gridDim.x + 1] offsets into units
    int heads;
    long long stride_b, stride_h, stride_s;  // elements
    __nv_bfloat16 *out;
    float scale_log2;
    int out_align32;
    const int *out_map;      // nullptr, or physical row -> row of `out` (fused exit gather)
    float *lse;              // nullptr, or [batch * heads, S]
    int S;
    int *status;
};

__device__ __forceinline__ int blocks_of(int len) { return (len + BN - 1) / BN; }

// first key row of the item's block `blk` (blocks are numbered through the ranges in order)
__device__ __forceinline__ int block_row(const WorkItem &it, int blk) {
    int row = 0;
#pragma unroll
    for (int s = 0; s < 3; ++s) {
        if (s < it.n_seg) {
            const int nb = blocks_of(it.seg_len[s]);
            if (blk >= 0 && blk < nb) row = it.seg_start[s] + blk * BN;
            blk -= nb;
        }
    }
    return row;
}

__global__ void __launch_bounds__(THREADS, 1)
attn_bf16_solo_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, const SoloParams prm) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[NUM_BARS];
    __shared__ float sh_m[2][BM], sh_a[2][BM];        // published by group w: reference maximum, rescale factor
    __shared__ float sh_l[2][BM], sh_f[2][BM];        // posted by group w: row sum, rounding correction
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ long long stamp[2];

    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sQ = smem_u32(smem);
    const uint32_t sKV = sQ + 2 * Q_BYTES;
    const int tid = threadIdx.x, warp = tid >> 5;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < NUM_BARS; ++i) {
            uint32_t count = 1;
            if (i >= S_FREE && i < S_FREE + 2) count = 4;
            if (i >= P_READY && i < P_READY + 4) count = 4;
            if (i == O_FREE) count = 4;
            if (i >= PUB && i < DRAIN) count = 1;   // one arrival per warp (its elected lane, after a warp sync)
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

    if (blockIdx.x == 0 && tid == 0) {
        // start stamps of the launch's first CTA (kept in shared memory: no register lives across the kernel)
        unsigned long long ns;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
        stamp[0] = clock64();
        stamp[1] = (long long)ns;
    }

    if (warp >= 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    }
    if (warp == 8) {
        // ------------------------------------------------------------ producer
        if (elect_one()) {
            prefetch_tmap(&tmQ);
            prefetch_tmap(&tmK);
            prefetch_tmap(&tmV);
            uint32_t e = 0;
            bool ok = true;
            // one ring entry: the K tile or the V tile of block `blk` of item `wi`
            auto emit = [&](bool is_v, const WorkItem &wi, int blk, int b, int h) {
                const uint32_t s = e % NSLOT, ph = (e / NSLOT) & 1;
                ++e;
                if (!wait_or_abort(bar(KV_EMPTY + s), ph ^ 1, &abort_flag, prm.status, 0x102)) return false;
                mbar_expect_tx(bar(KV_FULL + s), TILE_BYTES);
                const int row = block_row(wi, blk);
                const uint32_t dst = sKV + s * TILE_BYTES;
                // the block's 128 rows of K or V: two 64-column slabs
                const CUtensorMap *tm = is_v ? &tmV : &tmK;
#pragma unroll
                for (int sl = 0; sl < 2; ++sl)
                    tma_load_4d(dst + sl * (TILE_BYTES / 2), tm, bar(KV_FULL + s), 64 * sl, row, h, b);
                return true;
            };
            // The K tiles run two blocks ahead of the V tiles through ALL the CTA's items, in the
            // order the MMAs consume them: K(0) K(1) | K(2) V(0) | K(3) V(1) | ...  The query tile
            // of an item is requested just before its first K tile.
            int uk = u_begin, jk = 0;
            uint32_t uck = 0;
            WorkItem wk = {};
            int bk = 0, hk = 0;
            auto emit_next_k = [&]() {
                if (uk >= u_end) return true;
                if (jk == 0) {
                    const WorkUnit unit = prm.units[uk];
                    wk = prm.work[unit.item];
                    bk = unit.bh / prm.heads;
                    hk = unit.bh % prm.heads;
                    const uint32_t qb = uck & 1;
                    if (!wait_or_abort(bar(Q_EMPTY + qb), ((uck >> 1) & 1) ^ 1, &abort_flag, prm.status, 0x101))
                        return false;
                    mbar_expect_tx(bar(Q_FULL + qb), Q_BYTES);
#pragma unroll
                    for (int sl = 0; sl < 2; ++sl)
                        tma_load_4d(sQ + qb * Q_BYTES + sl * (Q_BYTES / 2), &tmQ, bar(Q_FULL + qb), 64 * sl, wk.q_start, hk, bk);
                }
                if (!emit(false, wk, jk, bk, hk)) return false;
                if (++jk == wk.kv_blocks) {
                    jk = 0;
                    ++uk;
                    ++uck;
                }
                return true;
            };
            ok = emit_next_k() && emit_next_k();
            for (int u = u_begin; ok && u < u_end; ++u) {
                const WorkUnit unit = prm.units[u];
                const WorkItem wi = prm.work[unit.item];
                const int b = unit.bh / prm.heads, h = unit.bh % prm.heads;
                for (int j = 0; ok && j < wi.kv_blocks; ++j) ok = emit_next_k() && emit(true, wi, j, b, h);
            }
            if (!ok) {
                // let every copy already issued land before the CTA retires
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000) {
                }
            }
        }
    } else if (warp == 9) {
        // ---------------------------------------------------------- MMA issuer
        if (elect_one()) {
            auto commit = [&](int i) { mma_commit(bar(i)); };
            constexpr uint32_t IDESC_QK = idesc_bf16_f32(BM, BN, 0, 0);
            constexpr uint32_t IDESC_PV = idesc_bf16_f32(BM, HD, 0, 1);
            uint32_t e = 0;
            bool ok = true;
            // S_b = Q K^T of the next block of the stream (launch-wide index Gq, buffer b = Gq & 1)
            int uq = u_begin, jq = 0, nq = 0;
            uint32_t Gq = 0, ucq = 0;
            auto issue_next_qk = [&]() {
                if (uq >= u_end) return true;
                const uint32_t qb = ucq & 1;
                if (jq == 0) {
                    nq = prm.work[prm.units[uq].item].kv_blocks;
                    if (!wait_or_abort(bar(Q_FULL + qb), (ucq >> 1) & 1, &abort_flag, prm.status, 0x201)) return false;
                }
                const uint32_t bf = Gq & 1;
                // the warpgroup has taken the scores of block Gq - 2 out of the buffer
                if (Gq >= 2 && !wait_or_abort(bar(S_FREE + bf), ((Gq >> 1) - 1) & 1, &abort_flag, prm.status, 0x202))
                    return false;
                const uint32_t s = e % NSLOT, ph = (e / NSLOT) & 1;
                ++e;
                if (!wait_or_abort(bar(KV_FULL + s), ph, &abort_flag, prm.status, 0x203)) return false;
                tc_fence_after();
                const uint64_t dq = smem_desc_sw128(sQ + qb * Q_BYTES, 16, 1024);
                const uint64_t dk = smem_desc_sw128(sKV + s * TILE_BYTES, 16, 1024);
#pragma unroll
                for (int k = 0; k < HD / 16; ++k) {
                    const uint64_t oq = (uint64_t)(((k >> 2) * (Q_BYTES / 2) + (k & 3) * 32) >> 4);
                    const uint64_t okk = (uint64_t)(((k >> 2) * (TILE_BYTES / 2) + (k & 3) * 32) >> 4);
                    mma_ss(tmem + COL_S + bf * BN, dq + oq, dk + okk, IDESC_QK, k > 0);
                }
                commit(S_FULL + bf);
                commit(KV_EMPTY + s);
                ++Gq;
                if (++jq == nq) {
                    commit(Q_EMPTY + qb);   // the item's last Q K^T has been issued
                    jq = 0;
                    ++uq;
                    ++ucq;
                }
                return true;
            };
            ok = issue_next_qk() && issue_next_qk();
            uint32_t G = 0, uc = 0;
            for (int u = u_begin; ok && u < u_end; ++u, ++uc) {
                const int n = prm.work[prm.units[u].item].kv_blocks;
                for (int j = 0; ok && j < n; ++j, ++G) {
                    ok = issue_next_qk();
                    if (!ok) break;
                    // O (+)= P_b V for block G
                    const uint32_t bf = G & 1;
                    const uint32_t s = e % NSLOT, ph = (e / NSLOT) & 1;
                    ++e;
                    ok = wait_or_abort(bar(KV_FULL + s), ph, &abort_flag, prm.status, 0x204);
                    if (!ok) break;
                    if (j == 0 && uc > 0) {
                        // the previous item's epilogue has read the accumulator
                        ok = wait_or_abort(bar(O_FREE), (uc - 1) & 1, &abort_flag, prm.status, 0x205);
                        if (!ok) break;
                    }
                    const uint64_t dv = smem_desc_sw128(sKV + s * TILE_BYTES, TILE_BYTES / 2, 1024);
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        ok = wait_or_abort(bar(P_READY + bf * 2 + half), (G >> 1) & 1, &abort_flag, prm.status,
                                           0x206 + half);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll
                        for (int k = 4 * half; k < 4 * half + 4; ++k)
                            mma_ts(tmem + COL_O, tmem + COL_P + bf * 64 + k * 8, dv + (uint64_t)((k * 2048) >> 4),
                                        IDESC_PV, (j > 0 || k > 0) ? 1u : 0u);
                    }
                    if (!ok) break;
                    commit(KV_EMPTY + s);
                    commit(PV_DONE + (G & 3));
                }
            }
            // every MMA issued above has retired before TMEM is released
            mma_commit(bar(DRAIN));
            wait_or_abort(bar(DRAIN), 0, &abort_flag, prm.status, 0x208);
        }
    } else if (warp < 8) {
        // ------------------------------------------------- softmax warpgroup w: blocks with G & 1 == w
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
        const uint32_t w = warp >> 2, q = warp & 3;
        const int r = tid & 127;
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        const uint32_t tS = tmem + lane_addr + COL_S + w * BN;
        const uint32_t tP = tmem + lane_addr + COL_P + w * 64;
        const uint32_t tO = tmem + lane_addr + COL_O;
        const float scale_log2 = prm.scale_log2;
        uint32_t G = 0;
        uint32_t cS = 0;      // blocks this group has taken
        uint32_t cC = 0;      // publications of the other group consumed
        uint32_t cPost = 0;   // row-sum posts this group has made
        uint32_t cSeen = 0;   // row-sum posts of the other group read
        uint32_t cCons = 0;   // end-of-item consumption notices waited for
        bool cons_pending = false;   // the item's last block has yet to consume this group's latest publication
        bool ok = true;
        auto arrive = [&](int i) { mbar_arrive(bar(i)); };
        // what the warp's lanes wrote to shared memory before is visible to whoever sees the arrival
        auto warp_arrive = [&](uint32_t b) {
            __syncwarp();
            if ((tid & 31) == 0) mbar_arrive(b);
        };
        for (int u = u_begin; ok && u < u_end; ++u) {
            const WorkUnit unit = prm.units[u];
            const WorkItem wi = prm.work[unit.item];
            const int n = wi.kv_blocks;
            float m_ref = 0.f, l = 0.f;
            float l_fix = 0.f;   // rounding errors of the blocks' largest weights: part of the output's normaliser, not of lse
            float alpha = 1.f;   // factor by which this group's latest block rescaled what was accumulated before it
            int j = 0;
            for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                const int nb = blocks_of(wi.seg_len[seg]);
                for (int jb = 0; ok && jb < nb; ++jb, ++j) {
                    const uint32_t Gb = G + (uint32_t)j;
                    if ((Gb & 1) != w) continue;
                    const int valid = min(BN, wi.seg_len[seg] - jb * BN);
                    ok = wait_or_abort(bar(S_FULL + w), cS & 1, &abort_flag, prm.status, 0x301 + w);
                    if (!ok) break;
                    ++cS;
                    tc_fence_after();
                    uint32_t s[BN];
#pragma unroll
                    for (int c = 0; c < BN / 32; ++c) tmem_ld32(tS + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
                    tmem_wait_ld();
                    // the scores are in registers: Q K^T of block G + 2 may overwrite the buffer
                    tc_fence_before();
                    __syncwarp();
                    if ((tid & 31) == 0) arrive(S_FREE + w);
                    if (valid < BN) {
#pragma unroll
                        for (int i = 0; i < BN; ++i)
                            if (i >= valid) s[i] = 0xff800000u;  // -inf
                    }
                    // Eight independent max chains, then a short tree.  Chain c takes the pairs of scores
                    // whose index is c modulo 8; with one pair in four on the polynomial (pairs 3 modulo
                    // 4) chains 3 and 7 see exactly the scores whose exponentials the FMA pipes will
                    // compute, the other six those of the MUFU unit, so the block maximum comes with the
                    // path its weight will take.
                    constexpr int PM = HB_POLY_MASK;
                    static_assert(PM == 3 || PM == 0xff, "the chain seeding below assumes pairs 3 mod 4 (or none) on the polynomial");
                    float mxa[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) mxa[i] = __uint_as_float(s[i == 3 ? 6 : (i == 6 ? 3 : i)]);
#pragma unroll
                    for (int i = 8; i < BN; i += 2) {
                        const int c = (i >> 1) & 7;
                        mxa[c] = max3(mxa[c], __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
                    }
                    const float mx_fma = fmaxf(mxa[3], mxa[7]);
                    const float mx_mufu = fmaxf(max3(mxa[0], mxa[1], mxa[2]), max3(mxa[4], mxa[5], mxa[6]));
                    const float mx_raw = fmaxf(mx_fma, mx_mufu);
                    const bool top_on_fma = PM == 3 && mx_fma > mx_mufu;
                    const float mx = mx_raw * scale_log2;
                    alpha = 1.f;
                    if (j == 0) {
                        m_ref = mx;   // nothing accumulated yet
                    } else {
                        // what the other group published after block G - 1: the rows' reference maximum
                        // and the factor by which it rescaled everything accumulated before
                        ok = wait_or_abort(bar(PUB + (w ^ 1) * 4 + q), cC & 1, &abort_flag, prm.status, 0x311);
                        if (!ok) break;
                        ++cC;
                        m_ref = sh_m[w ^ 1][r];
                        const float a = sh_a[w ^ 1][r];
                        // the item's last block: the publishing group has moved on and may publish again
                        if (j + 1 == n) warp_arrive(bar(CONS + (w ^ 1) * 4 + q));
                        l *= a;
                        l_fix *= a;
                        if (__any_sync(0xffffffffu, mx > m_ref + RESCALE_THRESHOLD)) {
                            const float m_new = fmaxf(m_ref, mx);
                            alpha = ex2(m_ref - m_new);
                            m_ref = m_new;
                        }
                    }
                    if (j + 1 < n) {
                        // publish before any further work: the other group's next block waits for this
                        if (cons_pending) {
                            // the slot still holds what the previous item's last block had to read
                            ok = wait_or_abort(bar(CONS + w * 4 + q), cCons & 1, &abort_flag, prm.status, 0x312);
                            if (!ok) break;
                            ++cCons;
                            cons_pending = false;
                        }
                        sh_m[w][r] = m_ref;
                        sh_a[w][r] = alpha;
                        warp_arrive(bar(PUB + w * 4 + q));
                        cons_pending = j + 2 == n;
                    }
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
                        // everything accumulated so far (blocks up to G - 1) belongs to the old reference
                        const uint32_t Gp = Gb - 1;
                        ok = wait_or_abort(bar(PV_DONE + (Gp & 3)), (Gp >> 2) & 1, &abort_flag, prm.status, 0x303 + w);
                        if (!ok) break;
                        tc_fence_after();
                        l *= alpha;
                        l_fix *= alpha;
#pragma unroll
                        for (int c = 0; c < HD / 32; ++c) {
                            uint32_t o[32];
                            tmem_ld32(tO + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                            tmem_st32(tO + c * 32, o);
                        }
                    }
                    const float nm = -m_ref;
                    const float2 sc2 = make_float2(scale_log2, scale_log2), nm2 = make_float2(nm, nm);
                    float2 sum[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
                    // The row sum is taken over the fp32 weights; the P V MMA sees them rounded.  For the
                    // block's largest weight the rounding error is added to a separate sum, so that
                    // numerator and denominator round together where it matters; the weight is recomputed
                    // exactly as the loop below computes it (same fused multiply-add, same exponential).
                    {
                        const float xm = fmaf(mx_raw, scale_log2, nm);
                        const float pm_fma = ex2_poly1<HB_POLY_DEG>(xm);
                        const float pm = top_on_fma ? pm_fma : ex2(xm);
                        l_fix += __uint_as_float(pack_bf16(0.f, pm) & 0xffff0000u) - pm;
                    }
                    if (Gb >= 2) {
                        // P_w still feeds the P V of this group's previous block
                        const uint32_t Gp = Gb - 2;
                        ok = wait_or_abort(bar(PV_DONE + (Gp & 3)), (Gp >> 2) & 1, &abort_flag, prm.status, 0x305 + w);
                        if (!ok) break;
                    }
#pragma unroll
                    for (int c = 0; c < BN / 32; ++c) {
                        uint32_t pk[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[c * 32 + 2 * i]),
                                                                    __uint_as_float(s[c * 32 + 2 * i + 1])),
                                                        sc2, nm2);
                            float2 p;
                            if ((i & PM) == PM) {
                                p = ex2_poly2<HB_POLY_DEG>(x);
                            } else {
                                p.x = ex2(x.x);
                                p.y = ex2(x.y);
                            }
                            pk[i] = pack_bf16(p.x, p.y);
                            sum[i & 3] = __fadd2_rn(sum[i & 3], p);
                        }
                        tmem_st16(tP + c * 16, pk);
                        if (c & 1) {  // keys [64 (c >> 1), +64) are in TMEM
                            tmem_wait_st();
                            tc_fence_before();
                            __syncwarp();
                            if ((tid & 31) == 0) arrive(P_READY + w * 2 + (c >> 1));
                        }
                    }
                    const float2 sa = __fadd2_rn(__fadd2_rn(sum[0], sum[1]), __fadd2_rn(sum[2], sum[3]));
                    l += sa.x + sa.y;
                }
            }
            if (!ok) break;
            // ---- end of the item
            const uint32_t G_last = G + (uint32_t)n - 1;
            G += (uint32_t)n;
            if ((G_last & 1) != w) {
                // The other group takes the item's last block and writes the output: leave this
                // group's row sums (in the scale of its own latest block) where it finds them and go
                // on to the next item.  The slot is free once the previous post has been read.
                if (cPost > 0) {
                    ok = wait_or_abort(bar(ACK + w * 4 + q), (cPost - 1) & 1, &abort_flag, prm.status, 0x321);
                    if (!ok) break;
                }
                ++cPost;
                sh_l[w][r] = l;
                sh_f[w][r] = l_fix;
                warp_arrive(bar(POST + w * 4 + q));
                continue;
            }
            ok = wait_or_abort(bar(POST + (w ^ 1) * 4 + q), cSeen & 1, &abort_flag, prm.status, 0x322);
            if (!ok) break;
            ++cSeen;
            // the other group's sums predate this group's last block: they take its rescale factor
            const float l_all = l + alpha * sh_l[w ^ 1][r];
            const float f_all = l_fix + alpha * sh_f[w ^ 1][r];
            warp_arrive(bar(ACK + (w ^ 1) * 4 + q));
            ok = wait_or_abort(bar(PV_DONE + (G_last & 3)), (G_last >> 2) & 1, &abort_flag, prm.status, 0x307 + w);
            if (!ok) break;
            tc_fence_after();
            // epilogue: O / l -> bf16 -> global; rows beyond the item are dropped
            const int bh = unit.bh;
            const int b = bh / prm.heads, h = bh % prm.heads;
            const float inv = 1.f / (l_all + f_all);
            const bool row_ok = r < wi.q_rows;
            int out_row = wi.q_start + r;
            if (prm.out_map && row_ok) out_row = prm.out_map[out_row];
            __nv_bfloat16 *orow = prm.out + (long long)b * prm.stride_b + (long long)h * prm.stride_h +
                                  (long long)out_row * prm.stride_s;
            // m_ref and l are in the base-2 domain of the scaled logits: LSE = ln 2 * (m_ref + log2 l)
            if (prm.lse && row_ok)
                prm.lse[(long long)bh * prm.S + out_row] = 0.6931471805599453f * (m_ref + log2f(l_all));
            uint32_t o[HD];
#pragma unroll
            for (int c = 0; c < HD / 32; ++c) tmem_ld32(tO + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&o[c * 32]));
            tmem_wait_ld();
            // the accumulator is in registers: the next item's first P V may overwrite it
            tc_fence_before();
            __syncwarp();
            if ((tid & 31) == 0) arrive(O_FREE);
            if (row_ok) {
#pragma unroll
                for (int c = 0; c < HD / 32; ++c) {
                    uint32_t wv[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        wv[i] = pack_bf16(__uint_as_float(o[c * 32 + 2 * i]) * inv, __uint_as_float(o[c * 32 + 2 * i + 1]) * inv);
                    if (prm.out_align32) {
#pragma unroll
                        for (int i = 0; i < 16; i += 8) st_global_v8(orow + c * 32 + 2 * i, wv + i);
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; i += 4)
                            *reinterpret_cast<uint4 *>(orow + c * 32 + 2 * i) = make_uint4(wv[i], wv[i + 1], wv[i + 2], wv[i + 3]);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (blockIdx.x == 0 && tid == 0) {
        // elapsed SM cycles and nanoseconds of this CTA: the launch's effective SM clock
        unsigned long long ns;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
        prm.status[32] = (int)(clock64() - stamp[0]);
        prm.status[33] = (int)((long long)ns - stamp[1]);
    }
    if (warp == 8) {
        __syncwarp();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

std::mutex g_attr_mutex;
bool g_attr_done[64] = {};

}  // namespace

int make_tensor_map(CUtensorMap *m, const void *base, const hilberta_plan_t *p, int box_rows, int heads);

// Work list (items of 128 rows) and the static schedule.
// Returns OK and leaves p->n_solo == 0 if this shape is not served by this kernel.
int attn_bf16_solo_prepare(hilberta_plan_t *p) {
    cudaFree(p->d_work_solo);
    cudaFree(p->d_units_solo);
    cudaFree(p->d_solo_begin);
    p->d_work_solo = nullptr;
    p->d_units_solo = nullptr;
    p->d_solo_begin = nullptr;
    p->n_solo = 0;
    if (p->dtype != HILBERTA_BF16 || p->head_dim != HD) return HILBERTA_OK;
    {
        // the shared-memory opt-in is a per-device attribute of the kernel
        std::lock_guard<std::mutex> lock(g_attr_mutex);
        if (p->device < 0 || p->device >= 64) return HILBERTA_ERR_INVALID;
        if (!g_attr_done[p->device]) {
            HB_CUDA(cudaFuncSetAttribute(attn_bf16_solo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
            g_attr_done[p->device] = true;
        }
    }
    auto cost_of = [](const WorkItem &it) { return (long long)it.kv_blocks * 10 + 6; };
    std::vector<WorkItem> items = build_work_items(p, ITEM_ROWS, BN);
    {
        const int rc_items = check_work_items(items.data(), (int)items.size(), p->S, ITEM_ROWS, BN);
        if (rc_items != HILBERTA_OK) return rc_items;
    }
    if (items.empty()) return HILBERTA_OK;
    std::stable_sort(items.begin(), items.end(),
                     [&](const WorkItem &a, const WorkItem &b) { return cost_of(a) > cost_of(b); });
    std::vector<long long> cost;
    for (const WorkItem &it : items) cost.push_back(cost_of(it));
    HB_CUDA(cudaMalloc(&p->d_work_solo, sizeof(WorkItem) * items.size()));
    HB_CUDA(cudaMemcpy(p->d_work_solo, items.data(), sizeof(WorkItem) * items.size(), cudaMemcpyHostToDevice));
    return upload_schedule(items, cost, p->batch * p->heads, p->sm_count, &p->d_units_solo, &p->d_solo_begin, &p->n_solo);
}

int launch_attn_bf16_solo(const hilberta_plan_t *p, const void *q, const void *k, const void *v, void *out,
                          float *lse, const int *out_map, cudaStream_t stream) {
    CUtensorMap mq, mk, mv;
    int rc;
    if ((rc = make_tensor_map(&mq, q, p, BM, p->heads)) != HILBERTA_OK) return rc;
    if ((rc = make_tensor_map(&mk, k, p, BN, p->heads)) != HILBERTA_OK) return rc;
    if ((rc = make_tensor_map(&mv, v, p, BN, p->heads)) != HILBERTA_OK) return rc;
    SoloParams prm;
    prm.work = p->d_work_solo;
    prm.units = p->d_units_solo;
    prm.cta_begin = p->d_solo_begin;
    prm.heads = p->heads;
    prm.stride_b = p->stride_b;
    prm.stride_h = p->stride_h;
    prm.stride_s = p->stride_s;
    prm.out = (__nv_bfloat16 *)out;
    prm.scale_log2 = p->scale * 1.4426950408889634f;
    prm.status = p->d_status;
    prm.out_map = out_map;
    prm.lse = lse;
    prm.S = p->S;
    prm.out_align32 = (((uintptr_t)out & 31) == 0 && ((p->stride_b | p->stride_h | p->stride_s) & 15) == 0) ? 1 : 0;
    attn_bf16_solo_kernel<<<p->n_solo, THREADS, SMEM_BYTES, stream>>>(mq, mk, mv, prm);
    HB_LAUNCHED();
    return HILBERTA_OK;
}

}  // namespace hilberta
