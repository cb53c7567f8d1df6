// Internal definitions shared by the library's translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "hilberta.h"

namespace hilberta {

extern thread_local int g_last_cuda_error;
extern std::atomic<uint64_t> g_launches;

#define HB_CUDA(expr)                                  \
    do {                                               \
        cudaError_t e__ = (expr);                      \
        if (e__ != cudaSuccess) {                      \
            ::hilberta::g_last_cuda_error = (int)e__;  \
            return HILBERTA_ERR_CUDA;                  \
        }                                              \
    } while (0)

#define HB_LAUNCHED()                                  \
    do {                                               \
        ::hilberta::g_launches.fetch_add(1);           \
        HB_CUDA(cudaGetLastError());                   \
    } while (0)

// One slid tile of the partition (Sec. 3.2) in physical coordinates: the
// non-shared members of Hilbert interval [lo, lo + tile) mod HW occupy seg0
// (the part starting at lo) and, if the interval wraps, seg1.
struct Window {
    int lo;
    int seg0_start, seg0_len;
    int seg1_start, seg1_len;
};

// One unit of work of the tensor-core kernel: up to `rows` consecutive physical
// query rows that share one key list of up to three contiguous ranges
// (prefix, seg0, seg1; or the whole sequence for prefix rows).
struct WorkItem {
    int q_start;
    int q_rows;
    int n_seg;
    int seg_start[3];
    int seg_len[3];
    int kv_blocks;  // sum over ranges of ceil(len / 128)
};

// A work item applied to one (batch, head).  Units are assigned to CTAs on the
// host (longest-processing-time-first) and stored grouped by CTA.  bh2 >= 0 (forward kernel
// only, items of one query tile): the same item for a second (batch, head), which takes the
// CTA's other query-tile slot with a K/V stream of its own.
struct WorkUnit {
    int item;
    int bh;
    int bh2;
};

}  // namespace hilberta

struct hilberta_plan_s {
    int device;
    int H, W, HW, k_log2;   // image grid; padded side n = 2^k_log2 >= max(H, W); HW = number of grid cells
    int frames, shared_frames;  // video volume: frames x H x W cells on a 3-D curve (frames == 1: an image)
    int ka_log2, kb_log2;       // video: frame axis padded to 2^ka, image axes to 2^kb
    int NP;                 // n * n: length of the padded Hilbert curve the tiles are cut on
    bool compact;           // tiles are equal groups over the non-shared tokens (Algorithm 1) instead of curve intervals
    int tile, offset, shared_region, n_text, n_shared, T, S, P;
    uint64_t nnz;
    // device tables
    int *d_hil_d2t, *d_hil_t2d;      // [HW]
    int *d_c;                        // [NP + 1] real non-shared cells with padded Hilbert index below d
    int *d_phys2orig, *d_orig2phys;  // [S]
    int *d_row_window;               // [S] window id of a physical row, -1 for prefix rows
    hilberta::Window *d_windows;     // [T]
    // host mirrors of the small tables
    std::vector<hilberta::Window> h_windows;
    std::vector<int> h_shared_runs;  // (start, len) pairs
    // binding
    bool bound;
    int batch, heads, head_dim, dtype;
    int64_t stride_b, stride_h, stride_s;
    float scale;
    hilberta::WorkItem *d_work;
    int n_work;
    hilberta::WorkUnit *d_units;  // [n_work * batch * heads], grouped by CTA
    int *d_cta_begin;             // [n_cta + 1]
    int n_cta;
    // a second schedule over a slice of chunk_heads heads (all batches), for the host-buffer entry
    // point, which pipelines copies and launches slice by slice; chunk_heads == heads: no slicing
    int chunk_heads;
    hilberta::WorkUnit *d_units_chunk;
    int *d_cta_begin_chunk;
    int n_cta_chunk;
    // the pair kernel's work list and schedule (bf16, head dim 128): items of 256 rows, one per
    // pair of SMs; n_pair == 0: the shape is served by the single-CTA kernel
    hilberta::WorkItem *d_work_pair;
    hilberta::WorkUnit *d_units_pair;
    int *d_pair_begin;
    int n_pair;
    // the one-tile kernel's work list and schedule (bf16, head dim 128): items of 128 rows
    hilberta::WorkItem *d_work_solo;
    hilberta::WorkUnit *d_units_solo;
    int *d_solo_begin;
    int n_solo;
    cudaStream_t s_in, s_out;           // copy streams of hilberta_forward_host (created on first use)
    std::vector<cudaEvent_t> ev_in, ev_done;
    // backward pass: 128-row items over the same key lists, their schedule, and the
    // per-row scratch delta = rowsum(dO * O) that both backward kernels read
    hilberta::WorkItem *d_bwd_work;
    int n_bwd_work;
    hilberta::WorkUnit *d_bwd_units;
    int *d_bwd_cta_begin;
    int n_bwd_cta;
    float *d_delta;               // [batch * heads * S]
    int *d_status;  // [4] error word + diagnostics written by bounded waits
    // workspace of hilberta_forward_host
    void *ws;
    size_t ws_bytes;
    int sm_count;
};

namespace hilberta {
// out_map: nullptr = write rows in physical order; else out_map[p] is the row of `out`
// that physical row p goes to (the exit gather fused into the epilogue).
// lse: nullptr, or [batch * heads, S] fp32 receiving log-sum-exp of the scaled logits
// (natural log), indexed like `out` rows.
// in_map: nullptr = q, k, v are in physical order; else they are in ORIGINAL order and physical
// row p is read from row in_map[p] (the entry gather fused into the loads).
// chunk: -1 = the whole bound problem; c >= 0 = heads [c * chunk_heads, (c + 1) * chunk_heads) of
// every batch item only (lse must be null then).
int launch_attn_fp32(const hilberta_plan_t *p, const void *q, const void *k, const void *v, void *out,
                     float *lse, const int *out_map, const int *in_map, cudaStream_t stream, int chunk = -1);
int launch_attn_bf16(const hilberta_plan_t *p, const void *q, const void *k, const void *v, void *out,
                     float *lse, const int *out_map, const int *in_map, cudaStream_t stream, int chunk = -1);
// schedule.cu: work lists (runs of item_rows rows with their up to three key ranges, counted in
// blocks of `block` rows) and the static longest-first assignment of (item, batch * head) units to CTAs
std::vector<WorkItem> build_work_items(const hilberta_plan_t *p, int item_rows, int block);
// HILBERTA_OK iff the list is safe to hand to a kernel (ranges inside [0, S), rows covered exactly once)
int check_work_items(const WorkItem *items, int n, int S, int item_rows, int block);
// the schedule on the host (see hilberta_schedule_units); returns the largest CTA load
long long build_schedule(int n_items, const long long *cost, const long long *cost_two_heads, int bh, int sm_count,
                         std::vector<WorkUnit> &units, std::vector<int> &cta_begin);
// cost_two_heads: nullptr, or per item the cost of running it for TWO (batch, head) indices in one unit
// (0: the item is not paired); such items are emitted as units of two consecutive indices.
int upload_schedule(const std::vector<WorkItem> &items, const std::vector<long long> &cost, int bh, int sm_count,
                    WorkUnit **d_units, int **d_cta_begin, int *n_cta_out,
                    const std::vector<long long> *cost_two_heads = nullptr);
int attn_bf16_prepare(hilberta_plan_t *p);
// attn_bf16_pair_sm100.cu: the forward kernel on pairs of SMs (bf16, head dim 128, inputs in physical order)
int attn_bf16_pair_prepare(hilberta_plan_t *p);
int launch_attn_bf16_pair(const hilberta_plan_t *p, const void *q, const void *k, const void *v, void *out,
                          float *lse, const int *out_map, cudaStream_t stream);
// attn_bf16_solo_sm100.cu: the forward kernel with one query tile per CTA and double-buffered scores
// (bf16, head dim 128, inputs in physical order)
int attn_bf16_solo_prepare(hilberta_plan_t *p);
int launch_attn_bf16_solo(const hilberta_plan_t *p, const void *q, const void *k, const void *v, void *out,
                          float *lse, const int *out_map, cudaStream_t stream);
int attn_bwd_prepare(hilberta_plan_t *p);
// dq, dk, dv (bf16, physical order, the bound strides) from dout, q, k, v, out and the forward's lse.
int launch_attn_bwd(const hilberta_plan_t *p, const void *dout, const void *q, const void *k, const void *v,
                    const void *out, const float *lse, void *dq, void *dk, void *dv, float *delta,
                    cudaStream_t stream);
int launch_attn_fp32_bwd(const hilberta_plan_t *p, const void *dout, const void *q, const void *k, const void *v,
                         const void *out, const float *lse, void *dq, void *dk, void *dv, float *delta,
                         cudaStream_t stream);
int launch_timeout_probe(const hilberta_plan_t *p, cudaStream_t stream);
// plan.cu: does a written tensor share a byte with another tensor of the bound layout?
bool bound_tensors_overlap(const hilberta_plan_t *p, const void *out, size_t esz_out, const void *in, size_t esz_in);
}  // namespace hilberta
