// bf16 block-sparse flash-attention forward for sm_100a (Algorithm 1, restated
// for Blackwell): TMA loads of contiguous Q / K / V tiles, tcgen05 MMAs with
// accumulators in tensor memory, fp32 online softmax, one launch for prefix
// rows and tile rows alike.
//
// A work item is up to 256 consecutive physical query rows (two 128-row query
// tiles) that share a key list of up to three contiguous ranges (prefix, tile
// range, wrapped tile range -- or the whole sequence for prefix rows).  The
// key list is cut into blocks of 128 keys; the ragged last block of a range is
// masked by column.  Prefix blocks and tile blocks run through one loop with
// one online-softmax state per row.
//
// Roles inside a CTA (one CTA per SM, persistent over work items):
//   warps 0-3  softmax + epilogue for query tile 0, thread r owns row r (TMEM lane r)
//   warps 4-7  softmax + epilogue for query tile 1
//   warp  8    TMA producer (one elected lane)
//   warp  9    MMA issuer   (one elected lane)
//   warps 10-11 idle (their registers go to the softmax warps, setmaxnreg); in the GATHER
//               instantiations they are the loaders that fetch tile rows through the permutation
// The two query tiles ping-pong: while one tile's softmax runs on the CUDA
// cores, the tensor cores work on the other tile's P V and next Q K^T.
// TMEM columns: S_t = Q_t K^T (fp32) at [128 t, 128 t + 128), overwritten in
// place by P_t (bf16, first 64 columns); O_t accumulators at [256 + 128 t, +128).
// The running maximum is only advanced when it grows by more than 2^8, so the
// O accumulator is rescaled rarely; exponentials stay below 2^8.
// Shared memory: two Q tiles, a ring of K / V tiles, and (TMA instantiations) 32 KB in which the
// softmax warps stage finished output rows, 4 KB per warp, for bulk tensor stores -- used where the
// output keeps the physical order; scattered output (fused exit gather) and warps with rows beyond
// the item store per lane.
// FP8 instantiations take q, k, v as e4m3 bytes (128-byte rows, one slab per tile), round the
// weights to e4m3 (four per TMEM column) and use kind::f8f6f4 MMAs; everything else is shared.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdlib>
#include <functional>
#include <mutex>
#include <queue>
#include <type_traits>
#include <utility>

#include "attn_softmax_math.cuh"
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace hilberta {
using namespace ptx;

namespace {

constexpr int BM = 128;        // rows per query tile
constexpr int BN = 128;        // keys per block
constexpr int QT = 2;          // query tiles per work item
constexpr int ITEM_ROWS = QT * BM;
constexpr int NSTAGE = 5;      // K/V ring slots at most (K0 V0 K1 V1 ...)
// Ring slots of an instantiation.  The TMA kernels stage their output rows in shared memory (32 KB:
// 4 KB per softmax warp) and store them with bulk tensor copies; with bf16 tiles of head dim 128 that
// space is the fifth ring slot, which this kernel does not miss (measured equal with four), while the
// gathering kernel does (40 % slower with four) and keeps five slots and per-lane stores.
__host__ __device__ constexpr int ring_slots(bool gather, int hd, bool fp8) { return (!gather && !fp8 && hd == 128) ? 4 : NSTAGE; }
constexpr int STAGE_BYTES = 8 * 4096;
constexpr int SLAB_BYTES = BN * 128;     // one 64-column slab of 128 rows (128-byte swizzled rows)
// bf16, head dim HD = 128: a tile is two slabs (32 KB); HD = 64: one slab (16 KB).
// e4m3 (fp8 = true), HD = 128: rows of 128 bytes, one slab.
__host__ __device__ constexpr int tile_bytes(int hd, bool fp8 = false) { return BN * hd * (fp8 ? 1 : 2); }
constexpr int THREADS = 384;   // 8 softmax warps + producer + MMA issuer + 2 idle (register donors)
__host__ __device__ constexpr int smem_bytes(int hd, bool fp8 = false, bool gather = false) {
    return (QT + ring_slots(gather, hd, fp8)) * tile_bytes(hd, fp8) + (gather ? 0 : STAGE_BYTES) + 1024;
}
constexpr uint32_t TMEM_COLS = 512;
constexpr float RESCALE_THRESHOLD = 8.0f;        // log2 units
// e4m3 weights: the running maximum may lag by 2^4 and every weight carries a factor 2^4 (divided
// out with the row sum at the end), so weights lie in (0, 2^8] under e4m3's largest value 448 and
// the smallest nonzero one, 2^-9, is 2^-13 of the reference maximum.
constexpr float RESCALE_THRESHOLD_FP8 = 4.0f;
constexpr float P_SHIFT_FP8 = 4.0f;
#ifndef HB_POLY_MASK_FP8
#define HB_POLY_MASK_FP8 HB_POLY_MASK
#endif
#ifndef HB_POLY_DEG_FP8
#define HB_POLY_DEG_FP8 2
#endif
#ifndef HB_HOST_SLICES
#define HB_HOST_SLICES 8   // hilberta_forward_host pipelines its copies and launches over about this many slices of heads
#endif
#ifndef HB_SPLIT_AT
#define HB_SPLIT_AT 2    // P goes to the MMA issuer in two parts: 32-key chunks 0..HB_SPLIT_AT, then the rest (2: 96 + 32 keys; measured 0.4-0.6 % faster than 64 + 64)
#endif
#ifndef HB_WARP_ARRIVE
#define HB_WARP_ARRIVE 0 // 1: one mbarrier arrival per softmax warp (after a warp sync) instead of one per thread; measured equal
#endif

enum Bar {
    Q_FULL = 0, Q_EMPTY, DRAIN,
    S_FULL,
    P_READY = S_FULL + QT,        // [t * 2 + part]: P columns of the keys of that part written, 128 arrivals
    PV_DONE = P_READY + 2 * QT,
    KV_FULL = PV_DONE + QT, KV_EMPTY = KV_FULL + NSTAGE,
    NUM_BARS = KV_EMPTY + NSTAGE
};

struct Params {
    const WorkItem *work;
    const WorkUnit *units;   // (item, batch*heads index), grouped by CTA
    const int *cta_begin;    // [gridDim.x + 1] offsets into units
    int heads;
    long long stride_b, stride_h, stride_s;  // elements
    __nv_bfloat16 *out;
    float scale_log2;
    int out_align32;         // out and its strides are 32-byte aligned: 32-byte stores allowed
    const int *out_map;      // nullptr, or physical row -> row of `out` (fused exit scatter)
    float *lse;              // nullptr, or [batch * heads, S] log-sum-exp (natural log), rows as `out`
    int S;
    int *status;
};

// Entry gather fused in (GATHER kernels): q, k, v are in ORIGINAL order and physical row p is read
// from row in_map[p].  Only the gathering kernel's parameter block carries these fields: growing the
// plain kernel's block changes its register allocation and costs it 1.5 %.
template <bool GATHER>
struct KernelParams : Params {};
template <>
struct KernelParams<true> : Params {
    const int *in_map;
    const void *gq, *gk, *gv;
};

__device__ __forceinline__ int item_blocks(const WorkItem &it, int seg) {
    return (it.seg_len[seg] + BN - 1) / BN;
}

// S_t = Q_t K^T for one 128-key block: HD / 16 MMAs of K = 16 (bf16) or HD / 32 of K = 32 (e4m3);
// either way an MMA consumes 32 bytes of every row.
template <int HD, bool FP8>
__device__ __forceinline__ void issue_qk(uint32_t tmem_s, uint32_t sQt, uint32_t sKslot) {
    // the start-address field is the low 14 bits (16-byte units): stepping K is one add
    const uint64_t dq = smem_desc_sw128(sQt, 16, 1024), dk = smem_desc_sw128(sKslot, 16, 1024);
    if constexpr (FP8) {
        constexpr uint32_t IDESC = idesc_e4m3_f32(BM, BN, 0);
#pragma unroll
        for (int k = 0; k < HD / 32; ++k) mma_ss_f8(tmem_s, dq + (uint64_t)((k * 32) >> 4), dk + (uint64_t)((k * 32) >> 4), IDESC, k > 0);
    } else {
        constexpr uint32_t IDESC = idesc_bf16_f32(BM, BN, 0, 0);
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) {
            const uint64_t off = (uint64_t)(((k >> 2) * SLAB_BYTES + (k & 3) * 32) >> 4);
            mma_ss(tmem_s, dq + off, dk + off, IDESC, k > 0);
        }
    }
}

// O_t (+)= P_t V for one 128-key block: P from TMEM, V row-major in smem (N-major operand).
// `part` 0 covers the keys of 32-key chunks 0..HB_SPLIT_AT, part 1 the rest.  A chunk is two MMAs of
// K = 16 (bf16: 8 columns of P and 16 rows of V each) or one of K = 32 (e4m3: 8 columns of P, four
// weights per column, and 32 rows of V).
template <int HD, bool FP8>
__device__ __forceinline__ void issue_pv_part(uint32_t tmem_o, uint32_t tmem_p, uint32_t sVslot, int part,
                                              bool accumulate) {
    const uint64_t dv = smem_desc_sw128(sVslot, SLAB_BYTES, 1024);
    constexpr int C1 = HB_SPLIT_AT + 1, C2 = BN / 32;
    static_assert(C1 >= 1 && C1 < C2, "both parts hold at least one chunk");
    if constexpr (FP8) {
        constexpr uint32_t IDESC = idesc_e4m3_f32(BM, HD, 1);
        if (part == 0) {
#pragma unroll
            for (int k = 0; k < C1; ++k)
                mma_ts_f8(tmem_o, tmem_p + k * 8, dv + (uint64_t)((k * 4096) >> 4), IDESC, (accumulate || k > 0) ? 1u : 0u);
        } else {
#pragma unroll
            for (int k = C1; k < C2; ++k) mma_ts_f8(tmem_o, tmem_p + k * 8, dv + (uint64_t)((k * 4096) >> 4), IDESC, 1u);
        }
    } else {
        constexpr uint32_t IDESC = idesc_bf16_f32(BM, HD, 0, 1);
        if (part == 0) {
#pragma unroll
            for (int k = 0; k < 2 * C1; ++k)
                mma_ts(tmem_o, tmem_p + k * 8, dv + (uint64_t)((k * 2048) >> 4), IDESC, (accumulate || k > 0) ? 1u : 0u);
        } else {
#pragma unroll
            for (int k = 2 * C1; k < 2 * C2; ++k) mma_ts(tmem_o, tmem_p + k * 8, dv + (uint64_t)((k * 2048) >> 4), IDESC, 1u);
        }
    }
}

constexpr int GATHER_THREADS = 64;  // warps 10 and 11

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

// GATHER = false: Q / K / V tiles arrive by TMA from tensors in physical order.
// GATHER = true : the tensors are in ORIGINAL order (the entry gather of Sec. 3.4 fused in): two loader
// warps fetch every tile row through the permutation table with 16-byte cp.async copies and place it
// where a 128-byte-swizzled TMA box would have put it, so everything downstream is unchanged.
// FP8: q, k, v hold e4m3 bytes (HD = 128 only); the weights P are rounded to e4m3 as well; out stays bf16.
template <bool GATHER, int HD, bool FP8 = false>
__global__ void __launch_bounds__(THREADS, 1)
attn_bf16_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                 const KernelParams<GATHER> prm) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[NUM_BARS];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ long long stamp[2];
    static_assert(!FP8 || HD == 128, "e4m3 operands: head dim 128 only");
#ifdef HB_STAMPS
    if (threadIdx.x == 0) {
        unsigned long long ns;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
        prm.status[1024 + 4 * blockIdx.x] = (int)(ns & 0x7fffffff);
    }
#endif
    constexpr int TILE_BYTES = tile_bytes(HD, FP8);
    constexpr int NS = ring_slots(GATHER, HD, FP8);
    constexpr int NSLAB = TILE_BYTES / SLAB_BYTES;
    using elem_t = typename std::conditional<FP8, uint8_t, __nv_bfloat16>::type;
    constexpr int EPC = 16 / (int)sizeof(elem_t);   // elements per 16-byte chunk

    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sQ = smem_u32(smem);
    const uint32_t sKV = sQ + QT * TILE_BYTES;
    const uint32_t sStage = sKV + NS * TILE_BYTES;   // TMA kernels only: 4 KB per softmax warp
    const int tid = threadIdx.x, warp = tid >> 5;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < NUM_BARS; ++i)
        {
            uint32_t count = 1;
            if (i >= P_READY && i < P_READY + 2 * QT) count = HB_WARP_ARRIVE ? 4 : 128;
            if (GATHER && (i == Q_FULL || (i >= KV_FULL && i < KV_FULL + NSTAGE))) count = GATHER_THREADS;
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

    // Registers move from the data-movement warpgroup to the two softmax warpgroups.  The split
    // is tuned: spills in the MMA issuer (fewer than 88) or in the softmax warps (fewer than
    // 208) both cost more than 5 % of the kernel time.
    if (warp >= 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
    }
    if constexpr (GATHER) {
    if (warp == 10 || warp == 11) {
        // ------------------------------------------------- gathering loaders (entry permute fused in)
        uint32_t kvc = 0, qc = 0;
        bool ok = true;
        // The stage's barrier counts one arrival per loader thread; each arrival fires by itself
        // when that thread's copies into the stage have landed, so the loaders never wait for data.
        auto publish = [&](uint32_t b) {
            asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(b) : "memory");
        };
        // Warp w of the two copies rows [64 w, 64 w + 64) of a tile, RPI adjacent rows per
        // instruction (16 bytes per lane; a row is CH = HD / 8 lanes wide).  Lane L fetches the
        // table entries of rows L and 32 + L of that range once per tile; the lanes that copy a
        // row pick its entry up by shuffle, so the table costs one load latency per tile.
        constexpr int CH = HD / EPC, RPI = 32 / CH;
        const int lane = tid & 31, chunk = lane % CH, sub = lane / CH, wrow = (warp - 10) * 64;
        const uint32_t dst_lane = (uint32_t)((chunk >> 3) * SLAB_BYTES + (wrow + sub) * 128);
        const int c7 = (chunk & 7) ^ sub;   // row & 7 = (RPI i + sub) & 7 = ((RPI i) & 7) ^ sub
        auto load_rows = [&](int row0, int &ia, int &ib) {
            const int pa = row0 + wrow + lane, pb = pa + 32;
            ia = pa < prm.S ? __ldg(prm.in_map + pa) : -1;   // rows beyond the sequence are
            ib = pb < prm.S ? __ldg(prm.in_map + pb) : -1;   // zero-filled, as TMA does
        };
        auto copy_tile = [&](uint32_t dst_tile, const elem_t *base, int ia, int ib) {
            const elem_t *src0 = base + chunk * EPC;
            const uint32_t dst0 = dst_tile + dst_lane;
#pragma unroll
            for (int i = 0; i < 64 / RPI; ++i) {
                const int orow = __shfl_sync(0xffffffffu, RPI * i < 32 ? ia : ib, ((RPI * i) & 31) + sub);
                const uint32_t dst = dst0 + i * (RPI * 128) + ((c7 ^ ((RPI * i) & 7)) << 4);
                cp_async16(dst, src0 + (long long)max(orow, 0) * prm.stride_s, orow >= 0 ? 16 : 0);
            }
        };
        for (int u = u_begin; ok && u < u_end; ++u) {
            const WorkUnit unit = prm.units[u];
            const WorkItem wi = prm.work[unit.item];
            const long long bh_off = (long long)(unit.bh / prm.heads) * prm.stride_b +
                                     (long long)(unit.bh % prm.heads) * prm.stride_h;
            const bool dual = unit.bh2 >= 0;   // the item for two heads, one per query-tile slot
            const long long bh_off2 = !dual ? bh_off
                                            : (long long)(unit.bh2 / prm.heads) * prm.stride_b +
                                                  (long long)(unit.bh2 % prm.heads) * prm.stride_h;
            const int nt = (dual || wi.q_rows > BM) ? 2 : 1;
            ok = wait_or_abort(bar(Q_EMPTY), (qc & 1) ^ 1, &abort_flag, prm.status, 0x111);
            if (!ok) break;
            ++qc;
            for (int t = 0; t < nt; ++t) {
                int ia, ib;
                load_rows(wi.q_start + (dual ? 0 : t * BM), ia, ib);
                copy_tile(sQ + t * TILE_BYTES, (const elem_t *)prm.gq + (t ? bh_off2 : bh_off), ia, ib);
            }
            publish(bar(Q_FULL));
            if (dual) {
                // two K/V streams (same rows, two heads), entries in the order the MMA issuer uses them:
                // K_0(0) K_1(0), then per block V_0(j) K_0(j+1) V_1(j) K_1(j+1)
                auto emit = [&](const void *g, long long off, int ia, int ib) {
                    const uint32_t sl = kvc % NSTAGE, ph = (kvc / NSTAGE) & 1;
                    ++kvc;
                    if (!wait_or_abort(bar(KV_EMPTY + sl), ph ^ 1, &abort_flag, prm.status, 0x112)) return false;
                    copy_tile(sKV + sl * TILE_BYTES, (const elem_t *)g + off, ia, ib);
                    publish(bar(KV_FULL + sl));
                    return true;
                };
                int ia, ib;
                load_rows(wi.seg_start[0], ia, ib);
                ok = emit(prm.gk, bh_off, ia, ib) && emit(prm.gk, bh_off2, ia, ib);
                for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                    const int nb = item_blocks(wi, seg);
                    for (int j = 0; ok && j < nb; ++j) {
                        int row_n = -1;
                        if (j + 1 < nb) row_n = wi.seg_start[seg] + (j + 1) * BN;
                        else if (seg + 1 < wi.n_seg) row_n = wi.seg_start[seg + 1];
                        int na = -1, nbi = -1;
                        if (row_n >= 0) load_rows(row_n, na, nbi);
                        ok = emit(prm.gv, bh_off, ia, ib);
                        if (row_n >= 0) ok = ok && emit(prm.gk, bh_off, na, nbi);
                        ok = ok && emit(prm.gv, bh_off2, ia, ib);
                        if (row_n >= 0) ok = ok && emit(prm.gk, bh_off2, na, nbi);
                        ia = na;
                        ib = nbi;
                    }
                }
                continue;
            }
            for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                const int nb = item_blocks(wi, seg);
                for (int j = 0; ok && j < nb; ++j) {
                    // the K and the V tile of a block share their rows: one pass copies both; the
                    // table entries are requested before the wait for the two free slots
                    int ia, ib;
                    load_rows(wi.seg_start[seg] + j * BN, ia, ib);
                    const uint32_t sk = kvc % NSTAGE, phk = (kvc / NSTAGE) & 1;
                    const uint32_t sv = (kvc + 1) % NSTAGE, phv = ((kvc + 1) / NSTAGE) & 1;
                    kvc += 2;
                    ok = wait_or_abort(bar(KV_EMPTY + sk), phk ^ 1, &abort_flag, prm.status, 0x112);
                    if (!ok) break;
                    ok = wait_or_abort(bar(KV_EMPTY + sv), phv ^ 1, &abort_flag, prm.status, 0x113);
                    if (!ok) break;
                    {
                        // one pass over the rows for both tiles: a shuffle and an address per row pair
                        const elem_t *k0 = (const elem_t *)prm.gk + bh_off + chunk * EPC;
                        const elem_t *v0 = (const elem_t *)prm.gv + bh_off + chunk * EPC;
                        const uint32_t dk0 = sKV + sk * TILE_BYTES + dst_lane, dv0 = sKV + sv * TILE_BYTES + dst_lane;
#pragma unroll
                        for (int i = 0; i < 64 / RPI; ++i) {
                            const int orow = __shfl_sync(0xffffffffu, RPI * i < 32 ? ia : ib, ((RPI * i) & 31) + sub);
                            const uint32_t o = i * (RPI * 128) + ((c7 ^ ((RPI * i) & 7)) << 4);
                            const long long so = (long long)max(orow, 0) * prm.stride_s;
                            cp_async16(dk0 + o, k0 + so, orow >= 0 ? 16 : 0);
                            cp_async16(dv0 + o, v0 + so, orow >= 0 ? 16 : 0);
                        }
                    }
                    publish(bar(KV_FULL + sk));
                    publish(bar(KV_FULL + sv));
                }
            }
        }
        // every copy lands before the CTA retires
        asm volatile("cp.async.wait_all;" ::: "memory");
    }
    }
    if (!GATHER && warp == 8) {
        // ------------------------------------------------------------ producer
        if (elect_one()) {
            prefetch_tmap(&tmQ);
            prefetch_tmap(&tmK);
            prefetch_tmap(&tmV);
            uint32_t kvc = 0, qc = 0;
            bool ok = true;
            // one ring entry: the K or V tile at key row `row` of head (h, b)
            auto emit = [&](const CUtensorMap *tm, int row, int h, int b) {
                const uint32_t s = kvc % NS, ph = (kvc / NS) & 1;
                ++kvc;
                if (!wait_or_abort(bar(KV_EMPTY + s), ph ^ 1, &abort_flag, prm.status, 0x102)) return false;
                mbar_expect_tx(bar(KV_FULL + s), TILE_BYTES);
#pragma unroll
                for (int sl = 0; sl < NSLAB; ++sl)
                    tma_load_4d(sKV + s * TILE_BYTES + sl * SLAB_BYTES, tm, bar(KV_FULL + s), 64 * sl, row, h, b);
                return true;
            };
            for (int u = u_begin; ok && u < u_end; ++u) {
                const WorkUnit unit = prm.units[u];
                const WorkItem wi = prm.work[unit.item];
                const int bh = unit.bh;
                const int b = bh / prm.heads, h = bh % prm.heads;
                const bool dual = unit.bh2 >= 0;   // the item for two heads, one per query-tile slot
                const int b2 = dual ? unit.bh2 / prm.heads : b, h2 = dual ? unit.bh2 % prm.heads : h;
                const int nt = (dual || wi.q_rows > BM) ? 2 : 1;
                ok = wait_or_abort(bar(Q_EMPTY), (qc & 1) ^ 1, &abort_flag, prm.status, 0x101);
                if (!ok) break;
                ++qc;
                mbar_expect_tx(bar(Q_FULL), nt * TILE_BYTES);
                for (int t = 0; t < nt; ++t) {
#pragma unroll
                    for (int sl = 0; sl < NSLAB; ++sl)
                        tma_load_4d(sQ + t * TILE_BYTES + sl * SLAB_BYTES, &tmQ, bar(Q_FULL), 64 * sl,
                                    wi.q_start + (dual ? 0 : t * BM), t ? h2 : h, t ? b2 : b);
                }
                // Ring entries in the order the MMA issuer consumes them.  One stream (both tiles read
                // the same tiles): K(0) V(0) K(1) V(1) ...  Two streams: K_0(0) K_1(0), then per block
                // V_0(j) K_0(j+1) V_1(j) K_1(j+1).
                bool first_block = true;
                for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                    const int nb = item_blocks(wi, seg);
                    for (int j = 0; ok && j < nb; ++j) {
                        const int row = wi.seg_start[seg] + j * BN;
                        if (!dual) {
                            ok = emit(&tmK, row, h, b) && emit(&tmV, row, h, b);
                        } else {
                            // the next block's key row, if there is one
                            int row_n = -1;
                            if (j + 1 < nb) row_n = row + BN;
                            else if (seg + 1 < wi.n_seg) row_n = wi.seg_start[seg + 1];
                            if (first_block) ok = emit(&tmK, row, h, b) && emit(&tmK, row, h2, b2);
                            first_block = false;
                            ok = ok && emit(&tmV, row, h, b);
                            if (row_n >= 0) ok = ok && emit(&tmK, row_n, h, b);
                            ok = ok && emit(&tmV, row, h2, b2);
                            if (row_n >= 0) ok = ok && emit(&tmK, row_n, h2, b2);
                        }
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
    } else if (warp == 9) {
        // ---------------------------------------------------------- MMA issuer
        if (elect_one()) {
            uint32_t ent = 0;   // ring entries consumed so far (the producer fills them in the order they are used here)
            uint32_t qc = 0;
            uint32_t cP[QT] = {0, 0};
            bool ok = true;
#ifdef HB_TIMING
            long long tm_p = 0, tm_kv = 0, tm_start = clock64();
#endif
            auto slot_of = [](uint32_t e) { return e % NS; };
            auto phase_of = [](uint32_t e) { return (e / NS) & 1; };
            // O_t (+)= P_t V for block j of tile t (P arrives in two parts so the MMAs of the first overlap
            // the rest of the softmax), then S_t = Q_t K^T for the next block if there is one
            auto tile_turn = [&](int t, uint32_t eV, uint32_t eKn, bool accumulate, bool more) {
#ifdef HB_TIMING
                const long long tp0 = clock64();
#endif
                if (!wait_or_abort(bar(P_READY + t * 2), cP[t] & 1, &abort_flag, prm.status, 0x205 + t)) return false;
                tc_fence_after();
#ifdef HB_TIMING
                tm_p += clock64() - tp0;
#endif
                issue_pv_part<HD, FP8>(tmem + 256 + t * HD, tmem + t * BN, sKV + slot_of(eV) * TILE_BYTES, 0, accumulate);
#ifdef HB_TIMING
                const long long tp1 = clock64();
#endif
                if (!wait_or_abort(bar(P_READY + t * 2 + 1), cP[t] & 1, &abort_flag, prm.status, 0x205 + t)) return false;
                ++cP[t];
#ifdef HB_TIMING
                tm_p += clock64() - tp1;
#endif
                tc_fence_after();
                issue_pv_part<HD, FP8>(tmem + 256 + t * HD, tmem + t * BN, sKV + slot_of(eV) * TILE_BYTES, 1, true);
                mma_commit(bar(PV_DONE + t));
                if (more) {
                    issue_qk<HD, FP8>(tmem + t * BN, sQ + t * TILE_BYTES, sKV + slot_of(eKn) * TILE_BYTES);
                    mma_commit(bar(S_FULL + t));
                }
                return true;
            };
            for (int u = u_begin; ok && u < u_end; ++u) {
                const WorkUnit unit = prm.units[u];
                const WorkItem wi = prm.work[unit.item];
                const bool dual = unit.bh2 >= 0;
                const int nt = (dual || wi.q_rows > BM) ? 2 : 1;
                const int n = wi.kv_blocks;
                ok = wait_or_abort(bar(Q_FULL), qc & 1, &abort_flag, prm.status, 0x201);
                if (!ok) break;
                ++qc;
                // tiles written by cp.async (generic proxy) are read by the tensor core (async proxy)
                if (GATHER) fence_proxy_async_smem();
                if (dual) {
                    // two K/V streams, one per tile: every ring entry serves one tile and is released as
                    // soon as the MMAs that read it are issued
                    for (int t = 0; t < 2; ++t, ++ent) {
                        ok = wait_or_abort(bar(KV_FULL + slot_of(ent)), phase_of(ent), &abort_flag, prm.status, 0x202);
                        if (!ok) break;
                        if (GATHER) fence_proxy_async_smem();
                        tc_fence_after();
                        issue_qk<HD, FP8>(tmem + t * BN, sQ + t * TILE_BYTES, sKV + slot_of(ent) * TILE_BYTES);
                        mma_commit(bar(S_FULL + t));
                        mma_commit(bar(KV_EMPTY + slot_of(ent)));
                    }
                    if (!ok) break;
                    if (n == 1) mma_commit(bar(Q_EMPTY));
                    for (int j = 0; ok && j < n; ++j) {
                        const bool more = j + 1 < n;
                        for (int t = 0; t < 2; ++t) {
                            const uint32_t eV = ent, eKn = ent + 1;
                            ent += more ? 2 : 1;
                            ok = wait_or_abort(bar(KV_FULL + slot_of(eV)), phase_of(eV), &abort_flag, prm.status, 0x204);
                            if (!ok) break;
                            if (more) {
                                ok = wait_or_abort(bar(KV_FULL + slot_of(eKn)), phase_of(eKn), &abort_flag, prm.status, 0x203);
                                if (!ok) break;
                            }
                            if (GATHER) fence_proxy_async_smem();
                            ok = tile_turn(t, eV, eKn, j > 0, more);
                            if (!ok) break;
                            mma_commit(bar(KV_EMPTY + slot_of(eV)));
                            if (more) mma_commit(bar(KV_EMPTY + slot_of(eKn)));
                        }
                        if (ok && j + 2 == n) mma_commit(bar(Q_EMPTY));
                    }
                    continue;
                }
                // one K/V stream: K of block j is entry ent + 2 j, V is ent + 2 j + 1
                // S_t(0)
                ok = wait_or_abort(bar(KV_FULL + slot_of(ent)), phase_of(ent), &abort_flag, prm.status, 0x202);
                if (!ok) break;
                if (GATHER) fence_proxy_async_smem();
                tc_fence_after();
                for (int t = 0; t < nt; ++t) {
                    issue_qk<HD, FP8>(tmem + t * BN, sQ + t * TILE_BYTES, sKV + slot_of(ent) * TILE_BYTES);
                    mma_commit(bar(S_FULL + t));
                }
                mma_commit(bar(KV_EMPTY + slot_of(ent)));
                if (n == 1) mma_commit(bar(Q_EMPTY));
                for (int j = 0; j < n; ++j, ent += 2) {
                    const uint32_t eV = ent + 1, eKn = ent + 2;
                    const bool more = j + 1 < n;
#ifdef HB_TIMING
                    const long long tk0 = clock64();
#endif
                    if (more) {
                        ok = wait_or_abort(bar(KV_FULL + slot_of(eKn)), phase_of(eKn), &abort_flag, prm.status, 0x203);
                        if (!ok) break;
                    }
                    ok = wait_or_abort(bar(KV_FULL + slot_of(eV)), phase_of(eV), &abort_flag, prm.status, 0x204);
                    if (!ok) break;
                    if (GATHER) fence_proxy_async_smem();
#ifdef HB_TIMING
                    tm_kv += clock64() - tk0;
#endif
                    for (int t = 0; ok && t < nt; ++t) ok = tile_turn(t, eV, eKn, j > 0, more);
                    if (!ok) break;
                    mma_commit(bar(KV_EMPTY + slot_of(eV)));
                    if (more) {
                        mma_commit(bar(KV_EMPTY + slot_of(eKn)));
                        if (j + 2 == n) mma_commit(bar(Q_EMPTY));
                    }
                }
            }
            // every MMA issued above has retired before TMEM is released
            mma_commit(bar(DRAIN));
            wait_or_abort(bar(DRAIN), 0, &abort_flag, prm.status, 0x207);
#ifdef HB_TIMING
            atomicAdd(prm.status + 16, (int)(tm_p >> 4));
            atomicAdd(prm.status + 17, (int)(tm_kv >> 4));
            atomicAdd(prm.status + 19, (int)((clock64() - tm_start) >> 4));
            atomicMax(prm.status + 20, (int)((clock64() - tm_start) >> 4));
            atomicMin(prm.status + 21, -(int)((clock64() - tm_start) >> 4));
#endif
        }
    } else if (warp < 8) {
        // ------------------------------------------------- softmax + epilogue, tile t
        asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
        const int t = warp >> 2;
        const int r = tid & 127;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_addr + t * BN;
        const uint32_t tO = tmem + lane_addr + 256 + t * HD;
        const float scale_log2 = prm.scale_log2;
        uint32_t cS = 0, cPV = 0;
        bool ok = true;
#ifdef HB_STAMPS
        int st_b2 = 0, st_b1 = 0, st_items2 = 0, st_items1 = 0, st_prefix_blocks = 0;
#endif
#ifdef HB_TIMING
        long long tm_wait = 0, tm_soft = 0, tm_epi = 0, tm_mark = clock64(), tm_blocks = 0;
#endif
        for (int u = u_begin; ok && u < u_end; ++u) {
            const WorkUnit unit = prm.units[u];
            const WorkItem wi = prm.work[unit.item];
#ifdef HB_STAMPS
            const long long st_unit_t0 = clock64();
            if (tid == 0) {
                if (wi.q_rows > BM) { st_b2 += wi.kv_blocks; ++st_items2; } else { st_b1 += wi.kv_blocks; ++st_items1; }
                if (wi.n_seg == 1) st_prefix_blocks += wi.kv_blocks;
            }
#endif
            const bool dual = unit.bh2 >= 0;   // the item for two heads: tile slot 1 holds the same rows of head bh2
            if (wi.q_rows <= t * BM && !dual) continue;  // this tile is absent from the item
            const int bh = (dual && t) ? unit.bh2 : unit.bh;
            const int b = bh / prm.heads, h = bh % prm.heads;
            float m_ref = 0.f, l = 0.f;
            float l_fix = 0.f;   // rounding errors of the blocks' largest weights: part of the output's normaliser, not of lse
            bool first = true;
            for (int seg = 0; ok && seg < wi.n_seg; ++seg) {
                const int nb = item_blocks(wi, seg);
                for (int j = 0; j < nb; ++j) {
                    const int valid = min(BN, wi.seg_len[seg] - j * BN);
                    ok = wait_or_abort(bar(S_FULL + t), cS & 1, &abort_flag, prm.status, 0x301 + t);
                    if (!ok) break;
                    ++cS;
#ifdef HB_TIMING
                    { const long long now = clock64(); tm_wait += now - tm_mark; tm_mark = now; ++tm_blocks; }
#endif
                    tc_fence_after();
                    uint32_t s[BN];
#pragma unroll
                    for (int c = 0; c < BN / 32; ++c) tmem_ld32(tS + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
                    tmem_wait_ld();
                    if (valid < BN) {
#pragma unroll
                        for (int i = 0; i < BN; ++i)
                            if (i >= valid) s[i] = 0xff800000u;  // -inf
                    }
                    // Eight independent max chains, then a short tree.  Chain c takes the pairs of scores
                    // whose index is c modulo 8; with one pair in four on the polynomial (pairs 3 modulo
                    // 4) chains 3 and 7 see exactly the scores whose exponentials the FMA pipes will
                    // compute, the other six those of the MUFU unit -- the first eight scores seed the
                    // chains accordingly (scores 6, 7 are pair 3; score 3 is pair 1).  So the block
                    // maximum comes with the path its weight will take, at no cost.
                    constexpr int PM = FP8 ? HB_POLY_MASK_FP8 : HB_POLY_MASK;
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
                    const float mx_raw = fmaxf(mx_fma, mx_mufu);            // the block's largest score, unscaled
                    const bool top_on_fma = PM == 3 && mx_fma > mx_mufu;    // ... and who computes its weight
                    float mx = mx_raw * scale_log2;
                    if (first) {
                        m_ref = mx;
                        first = false;
                    } else if (__any_sync(0xffffffffu, mx > m_ref + (FP8 ? RESCALE_THRESHOLD_FP8 : RESCALE_THRESHOLD))) {
                        // the accumulator of the blocks so far belongs to the old reference
                        ok = wait_or_abort(bar(PV_DONE + t), (cPV - 1) & 1, &abort_flag, prm.status, 0x303 + t);
                        if (!ok) break;
                        tc_fence_after();
                        const float m_new = fmaxf(m_ref, mx);
                        const float alpha = ex2(m_ref - m_new);
                        m_ref = m_new;
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
                    const float nm = FP8 ? P_SHIFT_FP8 - m_ref : -m_ref;
                    const float2 sc2 = make_float2(scale_log2, scale_log2), nm2 = make_float2(nm, nm);
                    float2 sum[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
                    // The row sum is taken over the fp32 weights; the P V MMA sees them rounded.  For
                    // the block's largest weight -- the one that dominates a near-one-hot row -- the
                    // rounding error is added to the sum, so numerator and denominator round together
                    // where it matters.  The weight is recomputed here exactly as the loop below will
                    // compute it (same fused multiply-add, same exponential): the MUFU unit and the
                    // polynomial agree to 8e-5 only, and a weight next to a rounding tie that rounded
                    // one way here and the other way there would double the error instead of cancelling it.
                    {
                        const float xm = fmaf(mx_raw, scale_log2, nm);
                        const float pm_fma = ex2_poly1<FP8 ? HB_POLY_DEG_FP8 : HB_POLY_DEG>(xm);
                        const float pm = top_on_fma ? pm_fma : ex2(xm);
                        if constexpr (FP8) l_fix += round_e4m3(pm) - pm;
                        else l_fix += __uint_as_float(pack_bf16(0.f, pm) & 0xffff0000u) - pm;
                    }
#pragma unroll
                    for (int c = 0; c < BN / 32; ++c) {
                        uint32_t pk[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            // packed fp32x2 arithmetic: one instruction per pair of scores
                            const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[c * 32 + 2 * i]),
                                                                    __uint_as_float(s[c * 32 + 2 * i + 1])),
                                                        sc2, nm2);
                            float2 p;
                            if ((i & PM) == PM) {
                                p = ex2_poly2<FP8 ? HB_POLY_DEG_FP8 : HB_POLY_DEG>(x);  // a fixed share of the pairs runs on the FMA pipes
                            } else {
                                p.x = ex2(x.x);
                                p.y = ex2(x.y);
                            }
                            if constexpr (FP8) {
                                // four weights per column: pairs 2 i' and 2 i' + 1 share pk[i']
                                const uint32_t h = pack_e4m3x2(p.x, p.y);
                                if (i & 1) pk[i >> 1] |= h << 16;
                                else pk[i >> 1] = h;
                            } else {
                                pk[i] = pack_bf16(p.x, p.y);
                            }
                            sum[i & 3] = __fadd2_rn(sum[i & 3], p);
                        }
                        if constexpr (FP8) tmem_st8(tS + c * 8, pk);
                        else tmem_st16(tS + c * 16, pk);
                        if (c == HB_SPLIT_AT || c == BN / 32 - 1) {  // a part of P is complete in TMEM
                            tmem_wait_st();
                            tc_fence_before();
                            if (HB_WARP_ARRIVE) __syncwarp();
                            if (!HB_WARP_ARRIVE || (tid & 31) == 0) {
                                mbar_arrive(bar(P_READY + t * 2 + (c == BN / 32 - 1 ? 1 : 0)));
                            }
                        }
                    }
                    {
                        const float2 sa = __fadd2_rn(__fadd2_rn(sum[0], sum[1]), __fadd2_rn(sum[2], sum[3]));
                        l += sa.x + sa.y;
                    }
                    ++cPV;
#ifdef HB_TIMING
                    { const long long now = clock64(); tm_soft += now - tm_mark; tm_mark = now; }
#endif
                }
            }
            if (!ok) break;
            // epilogue: O / l -> bf16 -> global; rows beyond the item are dropped
            ok = wait_or_abort(bar(PV_DONE + t), (cPV - 1) & 1, &abort_flag, prm.status, 0x305 + t);
            if (!ok) break;
            tc_fence_after();
            const float inv = 1.f / (l + l_fix);
            const int row = dual ? r : t * BM + r;
            // each thread stores its own row, so writing it at its ORIGINAL position instead
            // of the physical one (the exit gather of Sec. 3.4 fused in) costs one index read
            int out_row = wi.q_start + row;
            if (prm.out_map && row < wi.q_rows) out_row = prm.out_map[out_row];
            __nv_bfloat16 *orow = prm.out + (long long)b * prm.stride_b + (long long)h * prm.stride_h +
                                  (long long)out_row * prm.stride_s;
            // m_ref and l are in the base-2 domain of the scaled logits: LSE = ln 2 * (m_ref + log2 l)
            if (prm.lse && row < wi.q_rows)
                prm.lse[(long long)bh * prm.S + out_row] =
                    0.6931471805599453f * (m_ref - (FP8 ? P_SHIFT_FP8 : 0.f) + log2f(l));
            // Rows through shared memory and one bulk tensor store per 64 columns and warp: the
            // per-lane stores below cost 6 % of the launch at 2048^2 (10 % with 16 tiles at 1024^2)
            // on the SM's load/store path.  Only where the output keeps the physical order and all
            // 32 rows of the warp belong to the item (a box store would write the others too).
            const int row0 = (dual ? 0 : t * BM) + (warp & 3) * 32;   // the warp's first row in the item
            const bool bulk_out = !GATHER && (prm.out_align32 & 2) && row0 + 32 <= wi.q_rows;
            if (bulk_out) {
                const int lane = tid & 31;
                const uint32_t slot = sStage + warp * 4096;
#pragma unroll
                for (int rd = 0; rd < HD / 64; ++rd) {
                    // the bulk store that last used the slot has read it
                    if (lane == 0) bulk_wait_group_read0();
                    __syncwarp();
#pragma unroll
                    for (int c2 = 0; c2 < 2; ++c2) {
                        uint32_t o[32];
                        tmem_ld32(tO + rd * 64 + c2 * 32, o);
                        tmem_wait_ld();
                        uint32_t w[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            w[i] = pack_bf16(__uint_as_float(o[2 * i]) * inv, __uint_as_float(o[2 * i + 1]) * inv);
                        // row `lane` of a 128-byte-swizzled box: 16-byte chunk k sits at k ^ (row & 7)
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            st_shared_v4(slot + lane * 128 + (((c2 * 4 + k) ^ (lane & 7)) << 4), w + 4 * k);
                    }
                    fence_proxy_async_smem();   // generic-proxy writes -> the bulk copy's reads
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_4d(&tmO, slot, 64 * rd, wi.q_start + row0, h, b);
                        bulk_commit_group();
                    }
                }
            } else
#pragma unroll
            for (int c = 0; c < HD / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(tO + c * 32, o);
                tmem_wait_ld();
                if (row < wi.q_rows) {
                    uint32_t w[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        w[i] = pack_bf16(__uint_as_float(o[2 * i]) * inv, __uint_as_float(o[2 * i + 1]) * inv);
                    if (prm.out_align32 & 1) {
                        // 32-byte stores fill whole sectors: half the store instructions and
                        // half the L1/L2 write requests of 16-byte stores
#pragma unroll
                        for (int i = 0; i < 16; i += 8)
                            st_global_v8(orow + c * 32 + 2 * i, w + i);
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; i += 4)
                            *reinterpret_cast<uint4 *>(orow + c * 32 + 2 * i) = make_uint4(w[i], w[i + 1], w[i + 2], w[i + 3]);
                    }
                }
            }
            tc_fence_before();
#ifdef HB_TIMING
            { const long long now = clock64(); tm_epi += now - tm_mark; tm_mark = now; }
#endif
#ifdef HB_STAMPS
            if (tid == 0 && blockIdx.x % 5 == 4 && blockIdx.x / 5 < 32 && u - u_begin < 16) {
                int *w = prm.status + 3072 + (blockIdx.x / 5) * 32 + (u - u_begin) * 2;
                w[0] = wi.kv_blocks | ((wi.q_rows > BM ? 2 : 1) << 16) | ((wi.n_seg == 1 ? 1 : 0) << 20) | (1 << 24);
                w[1] = (int)(clock64() - st_unit_t0);
            }
#endif
        }
#ifdef HB_STAMPS
        if (tid == 0) {
            int *w = prm.status + 2048 + 8 * blockIdx.x;
            w[0] = st_b2; w[1] = st_b1; w[2] = st_items2; w[3] = st_items1; w[4] = st_prefix_blocks;
        }
#endif
#ifdef HB_TIMING
        if ((tid & 127) == 0) {
            atomicAdd(prm.status + 8 + t * 4 + 0, (int)(tm_wait >> 4));
            atomicAdd(prm.status + 8 + t * 4 + 1, (int)(tm_soft >> 4));
            atomicAdd(prm.status + 8 + t * 4 + 2, (int)(tm_epi >> 4));
            atomicAdd(prm.status + 8 + t * 4 + 3, (int)tm_blocks);
        }
#endif
    }

    // the epilogue's bulk stores are complete before the CTA gives up its shared memory
    if (!GATHER && warp < 8 && (tid & 31) == 0) bulk_wait_group0();
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
#ifdef HB_STAMPS
    if (threadIdx.x == 0) {
        unsigned long long ns;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
        prm.status[1024 + 4 * blockIdx.x + 1] = (int)(ns & 0x7fffffff);
        prm.status[1024 + 4 * blockIdx.x + 2] = (int)(stamp[1] & 0x7fffffff);
    }
#endif
}

// Exercises the bounded wait on purpose: one warp waits, with a 1 ms deadline, on a
// barrier that nothing ever arrives on, records the expiry like the attention kernel
// does and returns normally.  Used by hilberta_selftest_timeout.
__global__ void timeout_probe_kernel(int *status) {
    __shared__ uint64_t never;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&never), 1);
        mbar_fence_init();
    }
    __syncthreads();
    wait_or_abort(smem_u32(&never), 0, &abort_flag, status, 0x7e57, 2000000ll);
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

}  // namespace

// [batch, heads, S, head_dim] with element strides -> 4-D map, box = 128 bytes of a row (64 bf16 or
// 128 e4m3 columns) x box_rows rows.
int make_tensor_map(CUtensorMap *m, const void *base, const hilberta_plan_t *p, int box_rows, int heads) {
    if (heads <= 0) heads = p->heads;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return HILBERTA_ERR_CUDA;
    const bool fp8 = p->dtype == HILBERTA_FP8_E4M3;
    const cuuint64_t esz = fp8 ? 1 : 2;
    cuuint64_t dims[4] = {(cuuint64_t)p->head_dim, (cuuint64_t)p->S, (cuuint64_t)heads, (cuuint64_t)p->batch};
    cuuint64_t strides[3] = {(cuuint64_t)p->stride_s * esz, (cuuint64_t)p->stride_h * esz, (cuuint64_t)p->stride_b * esz};
    cuuint32_t box[4] = {fp8 ? 128u : 64u, (cuuint32_t)box_rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(m, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
                     const_cast<void *>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error = (int)cudaErrorInvalidValue;
        return HILBERTA_ERR_CUDA;
    }
    return HILBERTA_OK;
}

namespace {

// The output (always bf16) as a 4-D map with boxes of 64 columns x 32 rows, for the bulk stores of the
// epilogue.  false: the layout does not qualify (base or a stride not a multiple of 16 bytes) and the
// kernel keeps its per-lane stores.
bool make_out_tensor_map(CUtensorMap *m, const void *out, const hilberta_plan_t *p, int heads) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    if (((uintptr_t)out & 15) != 0 || ((p->stride_b | p->stride_h | p->stride_s) & 7) != 0) return false;
    cuuint64_t dims[4] = {(cuuint64_t)p->head_dim, (cuuint64_t)p->S, (cuuint64_t)heads, (cuuint64_t)p->batch};
    cuuint64_t strides[3] = {(cuuint64_t)p->stride_s * 2, (cuuint64_t)p->stride_h * 2, (cuuint64_t)p->stride_b * 2};
    cuuint32_t box[4] = {64u, 32u, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(out), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int launch_timeout_probe(const hilberta_plan_t *p, cudaStream_t stream) {
    timeout_probe_kernel<<<1, 32, 0, stream>>>(p->d_status);
    HB_LAUNCHED();
    return HILBERTA_OK;
}

// Work list (items of two query tiles, key blocks of 128) and the static schedules.
int attn_bf16_prepare(hilberta_plan_t *p) {
    // Cost of a unit in twentieths of a two-tile key block (about 140 SM cycles), from per-unit cycle
    // counts of the kernel at 1024^2 and 2048^2: two tiles 2760 cycles per block + 5500; one tile --
    // nothing to overlap its softmax with the MMAs -- 2580 per block + 2600, i.e. hardly cheaper.
    auto cost_of = [](const WorkItem &it) {
        return it.q_rows > BM ? (long long)it.kv_blocks * 20 + 40 : (long long)it.kv_blocks * 19 + 20;
    };
    std::vector<WorkItem> items = build_work_items(p, ITEM_ROWS, BN);
    {
        const int rc_items = check_work_items(items.data(), (int)items.size(), p->S, ITEM_ROWS, BN);
        if (rc_items != HILBERTA_OK) return rc_items;
    }
    std::stable_sort(items.begin(), items.end(),
                     [&](const WorkItem &a, const WorkItem &b) { return cost_of(a) > cost_of(b); });
    std::vector<long long> cost, cost_two_heads;
    for (const WorkItem &it : items) {
        cost.push_back(cost_of(it));
        // An item of one query tile leaves the CTA's other tile slot idle; run it for two heads at
        // once instead (each slot with a K/V stream of its own): the price of a two-tile unit, plus
        // the second stream's tile loads.
        cost_two_heads.push_back(it.q_rows > BM ? 0 : (long long)it.kv_blocks * 21 + 40);
    }
    cudaFree(p->d_work);
    cudaFree(p->d_units);
    cudaFree(p->d_cta_begin);
    cudaFree(p->d_units_chunk);
    cudaFree(p->d_cta_begin_chunk);
    p->d_work = nullptr;
    p->d_units = nullptr;
    p->d_cta_begin = nullptr;
    p->d_units_chunk = nullptr;
    p->d_cta_begin_chunk = nullptr;
    p->n_cta_chunk = 0;
    p->n_work = (int)items.size();
    p->n_cta = 0;
    if (items.empty()) return HILBERTA_OK;

    HB_CUDA(cudaMalloc(&p->d_work, sizeof(WorkItem) * items.size()));
    HB_CUDA(cudaMemcpy(p->d_work, items.data(), sizeof(WorkItem) * items.size(), cudaMemcpyHostToDevice));
    int rc = upload_schedule(items, cost, p->batch * p->heads, p->sm_count, &p->d_units, &p->d_cta_begin, &p->n_cta,
                             &cost_two_heads);
    if (rc != HILBERTA_OK) return rc;
    // slice of heads for the pipelined host-buffer path: the largest divisor of `heads` not above heads / HB_HOST_SLICES (rounded up)
    p->chunk_heads = p->heads;
    for (int d = (p->heads + HB_HOST_SLICES - 1) / HB_HOST_SLICES; d >= 1; --d)
        if (p->heads % d == 0) {
            p->chunk_heads = d;
            break;
        }
    if (p->chunk_heads < p->heads) {
        rc = upload_schedule(items, cost, p->batch * p->chunk_heads, p->sm_count, &p->d_units_chunk, &p->d_cta_begin_chunk,
                             &p->n_cta_chunk, &cost_two_heads);
        if (rc != HILBERTA_OK) return rc;
    }
    {
        // The shared-memory opt-in is an attribute of the kernel ON ONE DEVICE: set it once for every
        // device a plan is bound on (a failure is reported, not remembered).
        static std::mutex attr_mutex;
        static bool attr_done[64] = {};
        std::lock_guard<std::mutex> lock(attr_mutex);
        if (p->device < 0 || p->device >= 64) return HILBERTA_ERR_INVALID;
        if (!attr_done[p->device]) {
            HB_CUDA(cudaFuncSetAttribute(attn_bf16_kernel<false, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(128)));
            HB_CUDA(cudaFuncSetAttribute(attn_bf16_kernel<true, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(128, false, true)));
            HB_CUDA(cudaFuncSetAttribute(attn_bf16_kernel<false, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(64)));
            HB_CUDA(cudaFuncSetAttribute(attn_bf16_kernel<true, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(64, false, true)));
            HB_CUDA(cudaFuncSetAttribute(attn_bf16_kernel<false, 128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(128, true)));
            HB_CUDA(cudaFuncSetAttribute(attn_bf16_kernel<true, 128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(128, true, true)));
            attr_done[p->device] = true;
        }
    }
    {
        const int rc_solo = attn_bf16_solo_prepare(p);
        if (rc_solo != HILBERTA_OK) return rc_solo;
    }
    return attn_bf16_pair_prepare(p);
}

int launch_attn_bf16(const hilberta_plan_t *p, const void *q, const void *k, const void *v, void *out,
                     float *lse, const int *out_map, const int *in_map, cudaStream_t stream, int chunk) {
    if (p->n_work == 0) return HILBERTA_OK;
    // bf16 with head dim 128 and inputs in physical order can also run on pairs of SMs
    // (attn_bf16_pair_sm100.cu) or with one query tile per CTA (attn_bf16_solo_sm100.cu).  Those kernels
    // are correct but measure slower than this one, so they are opt-in: the environment variable
    // HILBERTA_FORWARD_KERNEL=pair or =solo selects them (read once).
    static const bool use_pair = [] {
        const char *e = getenv("HILBERTA_FORWARD_KERNEL");
        return e && e[0] == 'p';
    }();
    if (use_pair && !in_map && chunk < 0 && p->n_pair > 0)
        return launch_attn_bf16_pair(p, q, k, v, out, lse, out_map, stream);
    static const bool use_solo = [] {
        const char *e = getenv("HILBERTA_FORWARD_KERNEL");
        return e && e[0] == 's';
    }();
    if (use_solo && !in_map && chunk < 0 && p->n_solo > 0)
        return launch_attn_bf16_solo(p, q, k, v, out, lse, out_map, stream);
    int heads = p->heads, n_cta = p->n_cta;
    const WorkUnit *units = p->d_units;
    const int *cta_begin = p->d_cta_begin;
    const bool fp8 = p->dtype == HILBERTA_FP8_E4M3;
    if (chunk >= 0 && p->chunk_heads < p->heads) {
        // a slice of heads: same strides, shifted base pointers, the slice's own schedule
        if (lse) return HILBERTA_ERR_INVALID;
        heads = p->chunk_heads;
        const long long off = (long long)chunk * heads * p->stride_h;   // elements
        const long long esz_in = fp8 ? 1 : 2;
        q = (const char *)q + off * esz_in;
        k = (const char *)k + off * esz_in;
        v = (const char *)v + off * esz_in;
        out = (__nv_bfloat16 *)out + off;
        units = p->d_units_chunk;
        cta_begin = p->d_cta_begin_chunk;
        n_cta = p->n_cta_chunk;
    }
    CUtensorMap mq, mk, mv;
    int rc;
    if ((rc = make_tensor_map(&mq, q, p, BN, heads)) != HILBERTA_OK) return rc;
    if ((rc = make_tensor_map(&mk, k, p, BN, heads)) != HILBERTA_OK) return rc;
    if ((rc = make_tensor_map(&mv, v, p, BN, heads)) != HILBERTA_OK) return rc;
    Params prm;
    prm.work = p->d_work;
    prm.units = units;
    prm.cta_begin = cta_begin;
    prm.heads = heads;
    prm.stride_b = p->stride_b;
    prm.stride_h = p->stride_h;
    prm.stride_s = p->stride_s;
    prm.out = (__nv_bfloat16 *)out;
    prm.scale_log2 = p->scale * 1.4426950408889634f;
    prm.status = p->d_status;
    prm.out_map = out_map;
    prm.lse = lse;
    prm.S = p->S;
    // bit 0: 32-byte stores allowed; bit 1: rows leave through bulk tensor stores (physical order only)
    prm.out_align32 = (((uintptr_t)out & 31) == 0 && ((p->stride_b | p->stride_h | p->stride_s) & 15) == 0) ? 1 : 0;
    CUtensorMap mo = mq;   // a valid map in any case; read only with bit 1 set
    if (!in_map && !out_map && make_out_tensor_map(&mo, out, p, heads)) prm.out_align32 |= 2;
    if (in_map) {
        KernelParams<true> gprm;
        static_cast<Params &>(gprm) = prm;
        gprm.in_map = in_map;
        gprm.gq = q;
        gprm.gk = k;
        gprm.gv = v;
        if (fp8)
            attn_bf16_kernel<true, 128, true><<<n_cta, THREADS, smem_bytes(128, true, true), stream>>>(mq, mk, mv, mo, gprm);
        else if (p->head_dim == 128)
            attn_bf16_kernel<true, 128><<<n_cta, THREADS, smem_bytes(128, false, true), stream>>>(mq, mk, mv, mo, gprm);
        else
            attn_bf16_kernel<true, 64><<<n_cta, THREADS, smem_bytes(64, false, true), stream>>>(mq, mk, mv, mo, gprm);
    } else {
        KernelParams<false> pprm;
        static_cast<Params &>(pprm) = prm;
        if (fp8)
            attn_bf16_kernel<false, 128, true><<<n_cta, THREADS, smem_bytes(128, true), stream>>>(mq, mk, mv, mo, pprm);
        else if (p->head_dim == 128)
            attn_bf16_kernel<false, 128><<<n_cta, THREADS, smem_bytes(128), stream>>>(mq, mk, mv, mo, pprm);
        else
            attn_bf16_kernel<false, 64><<<n_cta, THREADS, smem_bytes(64), stream>>>(mq, mk, mv, mo, pprm);
    }
    HB_LAUNCHED();
    return HILBERTA_OK;
}

}  // namespace hilberta
