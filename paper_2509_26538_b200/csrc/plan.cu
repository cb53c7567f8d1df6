// Hilbert LUT generator, physical permutation and per-tile key ranges (device
// kernels), plus the plan object's host-side life cycle and table export.
#include <cstdio>
#include <cstring>
#include <new>

#include "common.cuh"

namespace hilberta {

thread_local int g_last_cuda_error = 0;
std::atomic<uint64_t> g_launches{0};

// ---------------------------------------------------------------------------
// Sec. 3.1 + appendix on general shapes: one thread per cell of the padded n x n
// grid (n = 2^k, the smallest power-of-two square that holds the H x W grid).
// Walk the bit planes of (col, row) from the most significant one down; each
// plane contributes a quadrant digit and re-orients the remaining sub-square.
// The orientation (start at row 0 / col 0, end at row 0 / col n-1) is the one
// the library documents.  Every padded index gets a kind: padding (outside
// H x W), real, or real and inside the central shared square (Sec. 3.3).
// ---------------------------------------------------------------------------
enum : unsigned char { CELL_PAD = 0, CELL_REAL = 1, CELL_SHARED = 2 };

__device__ __forceinline__ int hilbert2d_index(int k, int row, int col) {
    const int n = 1 << k;
    int x = col, y = row;
    int d = 0;
    for (int s = n >> 1; s > 0; s >>= 1) {
        const int rx = (x & s) ? 1 : 0;
        const int ry = (y & s) ? 1 : 0;
        d += s * s * ((3 * rx) ^ ry);
        if (ry == 0) {
            if (rx == 1) {
                x = n - 1 - x;
                y = n - 1 - y;
            }
            const int t = x;
            x = y;
            y = t;
        }
    }
    return d;
}

__global__ void hilbert_lut_kernel(int k, int H, int W, int *__restrict__ cell_of_pd,
                                   int *__restrict__ pd_of_cell, unsigned char *__restrict__ kind_by_pd,
                                   int sh_r0, int sh_c0, int sh_side) {
    const int n = 1 << k;
    const int pc = blockIdx.x * blockDim.x + threadIdx.x;   // padded cell
    if (pc >= n * n) return;
    const int row = pc >> k, col = pc & (n - 1);
    const int d = hilbert2d_index(k, row, col);
    if (row < H && col < W) {
        const int cell = row * W + col;
        pd_of_cell[cell] = d;
        cell_of_pd[d] = cell;
        const bool sh = row >= sh_r0 && row < sh_r0 + sh_side && col >= sh_c0 && col < sh_c0 + sh_side;
        kind_by_pd[d] = sh ? CELL_SHARED : CELL_REAL;
    } else {
        cell_of_pd[d] = -1;
        kind_by_pd[d] = CELL_PAD;
    }
}

// Video volumes (Sec. 5, "Extension to Video Diffusion"): one thread per cell of the padded
// volume of 2^a frames by 2^b x 2^b pixels.  A clip is usually much shorter than a frame is wide
// (a < b): the image plane is cut into macro cells of 2^a x 2^a pixels visited in the order of the
// 2-D curve, and the 2^a-cube of cells above a macro cell is walked by a 3-D Hilbert curve:
// index = macro index * 8^a + index inside the cube.  With a >= b the whole volume is one cube of
// side 2^a.  The 3-D index comes from the coordinate -> index direction of Skilling's transpose
// construction with axes (frame, row, col): per level, from the top bit down, an inversion or an
// exchange against axis 0; then a Gray encoding across the axes; the index is the bit interleave
// of the three resulting words (frame word most significant).
__device__ __forceinline__ int hilbert3d_index(int k, int f, int row, int col) {
    if (k == 0) return 0;
    unsigned X0 = f, X1 = row, X2 = col;
    for (unsigned Q = 1u << (k - 1); Q > 1; Q >>= 1) {
        const unsigned Pm = Q - 1;
        if (X0 & Q) X0 ^= Pm;                 // axis 0 against itself: inversion only
        if (X1 & Q) {
            X0 ^= Pm;
        } else {
            const unsigned t = (X0 ^ X1) & Pm;
            X0 ^= t;
            X1 ^= t;
        }
        if (X2 & Q) {
            X0 ^= Pm;
        } else {
            const unsigned t = (X0 ^ X2) & Pm;
            X0 ^= t;
            X2 ^= t;
        }
    }
    X1 ^= X0;
    X2 ^= X1;
    unsigned t = 0;
    for (unsigned Q = 1u << (k - 1); Q > 1; Q >>= 1)
        if (X2 & Q) t ^= Q - 1;
    X0 ^= t;
    X1 ^= t;
    X2 ^= t;
    int d = 0;
    for (int b = k - 1; b >= 0; --b)
        d = (d << 3) | (int)(((X0 >> b) & 1) << 2 | ((X1 >> b) & 1) << 1 | ((X2 >> b) & 1));
    return d;
}

__global__ void hilbert3d_lut_kernel(int a, int b, int F, int H, int W, int *__restrict__ cell_of_pd,
                                     int *__restrict__ pd_of_cell, unsigned char *__restrict__ kind_by_pd,
                                     int sh_f0, int sh_r0, int sh_c0, int sh_side, int sh_frames) {
    const int side = a >= b ? a : b;         // log2 of the padded image side
    const int pc = blockIdx.x * blockDim.x + threadIdx.x;   // padded cell, frame-major
    if (pc >= (1 << (a + 2 * side))) return;
    const int f = pc >> (2 * side), row = (pc >> side) & ((1 << side) - 1), col = pc & ((1 << side) - 1);
    int d;
    if (a >= b) {
        d = hilbert3d_index(a, f, row, col);
    } else {
        const int m = (1 << a) - 1;
        d = (hilbert2d_index(b - a, row >> a, col >> a) << (3 * a)) + hilbert3d_index(a, f, row & m, col & m);
    }
    if (f < F && row < H && col < W) {
        const int cell = (f * H + row) * W + col;
        pd_of_cell[cell] = d;
        cell_of_pd[d] = cell;
        const bool sh = f >= sh_f0 && f < sh_f0 + sh_frames && row >= sh_r0 && row < sh_r0 + sh_side &&
                        col >= sh_c0 && col < sh_c0 + sh_side;
        kind_by_pd[d] = sh ? CELL_SHARED : CELL_REAL;
    } else {
        cell_of_pd[d] = -1;
        kind_by_pd[d] = CELL_PAD;
    }
}

// c_ns[d] = number of real non-shared cells with padded index below d, c_real[d] =
// number of real cells below d, for d in [0, NP].  Single block; each thread owns a
// contiguous slice.
__global__ void cell_scan_kernel(const unsigned char *__restrict__ kind_by_pd, int NP, int *__restrict__ c_ns,
                                 int *__restrict__ c_real) {
    __shared__ int warp_ns[32], warp_real[32];
    const int tid = threadIdx.x;
    const int nthr = blockDim.x;
    const int per = (NP + nthr - 1) / nthr;
    const int lo = min(tid * per, NP), hi = min(lo + per, NP);
    int l_ns = 0, l_real = 0;
    for (int d = lo; d < hi; ++d) {
        const unsigned char kd = kind_by_pd[d];
        l_ns += kd == CELL_REAL;
        l_real += kd != CELL_PAD;
    }
    int v_ns = l_ns, v_real = l_real;
    const int lane = tid & 31, warp = tid >> 5;
    for (int off = 1; off < 32; off <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, v_ns, off), b = __shfl_up_sync(0xffffffffu, v_real, off);
        if (lane >= off) {
            v_ns += a;
            v_real += b;
        }
    }
    if (lane == 31) {
        warp_ns[warp] = v_ns;
        warp_real[warp] = v_real;
    }
    __syncthreads();
    if (warp == 0) {
        int a = (lane < (nthr >> 5)) ? warp_ns[lane] : 0, b = (lane < (nthr >> 5)) ? warp_real[lane] : 0;
        for (int off = 1; off < 32; off <<= 1) {
            const int ta = __shfl_up_sync(0xffffffffu, a, off), tb = __shfl_up_sync(0xffffffffu, b, off);
            if (lane >= off) {
                a += ta;
                b += tb;
            }
        }
        warp_ns[lane] = a;   // inclusive over warps
        warp_real[lane] = b;
    }
    __syncthreads();
    int run_ns = v_ns - l_ns + (warp ? warp_ns[warp - 1] : 0);
    int run_real = v_real - l_real + (warp ? warp_real[warp - 1] : 0);
    for (int d = lo; d < hi; ++d) {
        c_ns[d] = run_ns;
        c_real[d] = run_real;
        const unsigned char kd = kind_by_pd[d];
        run_ns += kd == CELL_REAL;
        run_real += kd != CELL_PAD;
    }
    if (tid == nthr - 1) {  // the last thread's running totals are the grand totals
        c_ns[NP] = run_ns;
        c_real[NP] = run_real;
    }
}

// Appendix A layout: text first, then shared tokens, then the rest, each image
// group by ascending Hilbert index.  One thread per original token.  Also the
// rank tables (Hilbert index among the real cells <-> cell).
// compact_R > 0 selects the group arithmetic of Algorithm 1: tile ids follow the position
// in the non-shared sequence (c_ns) instead of the position on the padded curve.
__global__ void layout_kernel(int HW, int NP, int n_text, int P, int tile, int offset, int compact_R,
                              const int *__restrict__ pd_of_cell, const int *__restrict__ c_ns,
                              const int *__restrict__ c_real, const unsigned char *__restrict__ kind_by_pd,
                              int *__restrict__ hil_d2t, int *__restrict__ hil_t2d,
                              int *__restrict__ phys2orig, int *__restrict__ orig2phys,
                              int *__restrict__ row_window) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_text + HW) return;
    if (t < n_text) {
        phys2orig[t] = t;
        orig2phys[t] = t;
        row_window[t] = -1;
        return;
    }
    const int cell = t - n_text;
    const int d = pd_of_cell[cell];
    const int rank = c_real[d];
    hil_t2d[cell] = rank;
    hil_d2t[rank] = cell;
    const int below = c_ns[d];
    int phys;
    if (kind_by_pd[d] == CELL_SHARED) {
        phys = n_text + (rank - below);
        row_window[phys] = -1;
    } else {
        phys = P + below;
        row_window[phys] = compact_R > 0 ? ((below + offset) % compact_R) / tile : ((d + offset) % NP) / tile;
    }
    phys2orig[phys] = t;
    orig2phys[t] = phys;
}

// Sec. 3.2 with wrap-around: slid tile w covers (padded) Hilbert indices
// [w*tile - offset, +tile) mod NP; its real non-shared members are contiguous in
// the physical order, in one range or two if the interval wraps.
__global__ void window_kernel(int NP, int T, int tile, int offset, int P, const int *__restrict__ c,
                              Window *__restrict__ win) {
    const int w = blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= T) return;
    long long lo_ll = ((long long)w * tile - offset) % NP;
    if (lo_ll < 0) lo_ll += NP;
    const int lo = (int)lo_ll;
    const int hi = lo + tile;
    Window r;
    r.lo = lo;
    const int a0 = lo, b0 = hi <= NP ? hi : NP;
    const int n0 = c[b0] - c[a0];
    r.seg0_start = n0 > 0 ? P + c[a0] : 0;
    r.seg0_len = n0;
    r.seg1_start = 0;
    r.seg1_len = 0;
    if (hi > NP) {
        const int n1 = c[hi - NP] - c[0];
        r.seg1_start = n1 > 0 ? P + c[0] : 0;
        r.seg1_len = n1;
    }
    win[w] = r;
}

// Appendix A / Algorithm 1 read literally: `groups` equal groups of `size` tokens over
// the R non-shared tokens in curve order, slid by `offset` positions of that sequence.
__global__ void window_compact_kernel(int R, int groups, int size, int offset, int P, Window *__restrict__ win) {
    const int w = blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= groups) return;
    Window r;
    long long lo_ll = ((long long)w * size - offset) % R;
    if (lo_ll < 0) lo_ll += R;
    const int lo = (int)lo_ll;
    r.lo = lo;
    r.seg0_start = P + lo;
    r.seg0_len = lo + size <= R ? size : R - lo;
    r.seg1_start = lo + size <= R ? 0 : P;
    r.seg1_len = lo + size <= R ? 0 : lo + size - R;
    win[w] = r;
}

static void free_plan(hilberta_plan_t *p) {
    if (!p) return;
    cudaFree(p->d_hil_d2t);
    cudaFree(p->d_hil_t2d);
    cudaFree(p->d_c);
    cudaFree(p->d_phys2orig);
    cudaFree(p->d_orig2phys);
    cudaFree(p->d_row_window);
    cudaFree(p->d_windows);
    cudaFree(p->d_work);
    cudaFree(p->d_units);
    cudaFree(p->d_cta_begin);
    cudaFree(p->d_units_chunk);
    cudaFree(p->d_work_pair);
    cudaFree(p->d_units_pair);
    cudaFree(p->d_pair_begin);
    cudaFree(p->d_work_solo);
    cudaFree(p->d_units_solo);
    cudaFree(p->d_solo_begin);
    cudaFree(p->d_cta_begin_chunk);
    for (cudaEvent_t e : p->ev_in) cudaEventDestroy(e);
    for (cudaEvent_t e : p->ev_done) cudaEventDestroy(e);
    if (p->s_in) cudaStreamDestroy(p->s_in);
    if (p->s_out) cudaStreamDestroy(p->s_out);
    cudaFree(p->d_bwd_work);
    cudaFree(p->d_bwd_units);
    cudaFree(p->d_bwd_cta_begin);
    cudaFree(p->d_delta);
    cudaFree(p->d_status);
    cudaFree(p->ws);
    delete p;
}

static int build_plan(hilberta_plan_t *p) {
    const int HW = p->HW, S = p->S, NP = p->NP;
    unsigned char *d_kind = nullptr;
    int *d_cell_of_pd = nullptr, *d_pd_of_cell = nullptr, *d_c_real = nullptr;
    HB_CUDA(cudaMalloc(&p->d_hil_d2t, sizeof(int) * HW));
    HB_CUDA(cudaMalloc(&p->d_hil_t2d, sizeof(int) * HW));
    HB_CUDA(cudaMalloc(&p->d_c, sizeof(int) * (NP + 1)));
    HB_CUDA(cudaMalloc(&p->d_phys2orig, sizeof(int) * S));
    HB_CUDA(cudaMalloc(&p->d_orig2phys, sizeof(int) * S));
    HB_CUDA(cudaMalloc(&p->d_row_window, sizeof(int) * S));
    HB_CUDA(cudaMalloc(&p->d_windows, sizeof(Window) * p->T));
    HB_CUDA(cudaMalloc(&p->d_status, sizeof(int) * 4096));
    HB_CUDA(cudaMemset(p->d_status, 0, sizeof(int) * 4096));

    const int sh_r0 = p->H / 2 - p->shared_region / 2;
    const int sh_c0 = p->W / 2 - p->shared_region / 2;
    int rc = HILBERTA_OK;
    do {
        cudaError_t e = cudaMalloc(&d_kind, NP);
        if (e == cudaSuccess) e = cudaMalloc(&d_cell_of_pd, sizeof(int) * NP);
        if (e == cudaSuccess) e = cudaMalloc(&d_pd_of_cell, sizeof(int) * HW);
        if (e == cudaSuccess) e = cudaMalloc(&d_c_real, sizeof(int) * (NP + 1));
        if (e != cudaSuccess) {
            g_last_cuda_error = (int)e;
            rc = HILBERTA_ERR_CUDA;
            break;
        }
        if (p->frames > 1)
            hilbert3d_lut_kernel<<<(NP + 255) / 256, 256>>>(p->ka_log2, p->kb_log2, p->frames, p->H, p->W, d_cell_of_pd,
                                                            d_pd_of_cell, d_kind, p->frames / 2 - p->shared_frames / 2,
                                                            sh_r0, sh_c0, p->shared_region, p->shared_frames);
        else
            hilbert_lut_kernel<<<(NP + 255) / 256, 256>>>(p->k_log2, p->H, p->W, d_cell_of_pd, d_pd_of_cell, d_kind,
                                                          sh_r0, sh_c0, p->shared_region);
        g_launches.fetch_add(1);
        cell_scan_kernel<<<1, 1024>>>(d_kind, NP, p->d_c, d_c_real);
        g_launches.fetch_add(1);
        layout_kernel<<<(S + 255) / 256, 256>>>(HW, NP, p->n_text, p->P, p->tile, p->offset,
                                                p->compact ? S - p->P : 0, d_pd_of_cell, p->d_c,
                                                d_c_real, d_kind, p->d_hil_d2t, p->d_hil_t2d, p->d_phys2orig,
                                                p->d_orig2phys, p->d_row_window);
        g_launches.fetch_add(1);
        if (p->compact)
            window_compact_kernel<<<(p->T + 127) / 128, 128>>>(S - p->P, p->T, p->tile, p->offset, p->P, p->d_windows);
        else
            window_kernel<<<(p->T + 127) / 128, 128>>>(NP, p->T, p->tile, p->offset, p->P, p->d_c, p->d_windows);
        g_launches.fetch_add(1);
        e = cudaGetLastError();
        if (e == cudaSuccess) e = cudaDeviceSynchronize();
        if (e != cudaSuccess) {
            g_last_cuda_error = (int)e;
            rc = HILBERTA_ERR_CUDA;
            break;
        }
        // host mirrors of the small tables
        p->h_windows.resize(p->T);
        std::vector<unsigned char> h_kind(NP);
        e = cudaMemcpy(p->h_windows.data(), p->d_windows, sizeof(Window) * p->T, cudaMemcpyDeviceToHost);
        if (e == cudaSuccess) e = cudaMemcpy(h_kind.data(), d_kind, NP, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) {
            g_last_cuda_error = (int)e;
            rc = HILBERTA_ERR_CUDA;
            break;
        }
        int n_sh = 0;
        for (int d = 0; d < NP; ++d) {
            if (h_kind[d] != CELL_SHARED) continue;
            ++n_sh;
            size_t n = p->h_shared_runs.size();
            if (n && p->h_shared_runs[n - 2] + p->h_shared_runs[n - 1] == d) {
                p->h_shared_runs[n - 1] += 1;
            } else {
                p->h_shared_runs.push_back(d);
                p->h_shared_runs.push_back(1);
            }
        }
        if (n_sh != p->n_shared) {
            rc = HILBERTA_ERR_INVALID;  // cannot happen for validated arguments
            break;
        }
        // kept pairs: prefix rows see everything; other rows see the prefix and
        // the non-shared members of their own slid tile
        const uint64_t Pq = (uint64_t)p->P, Sq = (uint64_t)S;
        uint64_t nnz = Pq * Sq;
        for (const Window &w : p->h_windows) {
            const uint64_t r = (uint64_t)w.seg0_len + (uint64_t)w.seg1_len;
            nnz += r * (Pq + r);
        }
        p->nnz = nnz;
    } while (0);
    cudaFree(d_kind);
    cudaFree(d_cell_of_pd);
    cudaFree(d_pd_of_cell);
    cudaFree(d_c_real);
    return rc;
}

}  // namespace hilberta

using namespace hilberta;

// tile > 0: curve tiling (tiles of `tile` positions of the padded curve).
// groups > 0: compact tiling (Algorithm 1's equal groups over the non-shared tokens).
// frames > 1: a video volume of `frames` x H x W cells on the 3-D curve of the padded cube, with a
// central shared box of shared_frames x shared_region x shared_region cells.
static int make_plan(int frames, int H, int W, int tile, int groups, int layer_offset, int shared_region,
                     int shared_frames, int n_text, hilberta_plan_t **out) {
    if (!out) return HILBERTA_ERR_INVALID;
    *out = nullptr;
    const bool compact = groups > 0;
    if (frames < 1 || H < 1 || W < 1 || n_text < 0 || shared_region < 0 || shared_frames < 0)
        return HILBERTA_ERR_INVALID;
    if (!compact && tile < 1) return HILBERTA_ERR_INVALID;
    if (H > 1024 || W > 1024) return HILBERTA_ERR_UNSUPPORTED;
    if (frames > 1 && (H > 128 || W > 128 || frames > 128)) return HILBERTA_ERR_UNSUPPORTED;
    const int HW = frames * H * W;        // grid cells = image (or video) tokens
    int k_log2 = 0;                       // padded image side n = 2^k >= max(H, W)
    while ((1 << k_log2) < (H > W ? H : W)) ++k_log2;
    int ka = 0, kb = k_log2;              // video: frames padded to 2^ka, image axes to 2^kb
    int NP = 1 << (2 * k_log2);           // length of the padded curve
    if (frames > 1) {
        ka = 1;
        while ((1 << ka) < frames) ++ka;
        if (ka >= kb) {                   // one cube of side 2^ka
            k_log2 = ka;
            NP = 1 << (3 * ka);
        } else {                          // macro cells of 2^ka x 2^ka pixels under cubes of side 2^ka
            NP = 1 << (2 * kb + ka);
        }
    }
    if (shared_region % 2 || shared_region > H || shared_region > W) return HILBERTA_ERR_INVALID;
    if (frames > 1) {
        if (shared_frames % 2 || shared_frames > frames) return HILBERTA_ERR_INVALID;
        if ((shared_frames == 0) != (shared_region == 0)) return HILBERTA_ERR_INVALID;  // a box needs both extents
    } else {
        shared_frames = 1;
    }
    if ((long long)n_text + HW > (1ll << 30)) return HILBERTA_ERR_INVALID;
    const int n_shared = shared_region * shared_region * shared_frames;
    const int R = HW - n_shared;          // non-shared image tokens
    if (compact) {
        if (R < 1 || R % groups) return HILBERTA_ERR_INVALID;
        tile = R / groups;
    } else if (NP % tile) {
        return HILBERTA_ERR_INVALID;
    }

    int dev = 0;
    HB_CUDA(cudaGetDevice(&dev));
    cudaDeviceProp prop;
    HB_CUDA(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return HILBERTA_ERR_ARCH;

    hilberta_plan_t *p = new (std::nothrow) hilberta_plan_t();
    if (!p) return HILBERTA_ERR_NOMEM;
    p->device = dev;
    p->sm_count = prop.multiProcessorCount;
    p->frames = frames;
    p->shared_frames = frames > 1 ? shared_frames : 0;
    p->H = H;
    p->W = W;
    p->HW = HW;
    p->NP = NP;
    p->k_log2 = k_log2;
    p->ka_log2 = ka;
    p->kb_log2 = kb;
    p->compact = compact;
    p->tile = tile;
    const long long period = compact ? R : NP;
    long long o = (long long)layer_offset % period;
    if (o < 0) o += period;
    p->offset = (int)o;
    p->shared_region = shared_region;
    p->n_text = n_text;
    p->n_shared = n_shared;
    p->T = compact ? groups : NP / tile;
    p->S = n_text + HW;
    p->P = n_text + p->n_shared;
    p->bound = false;
    int rc = build_plan(p);
    if (rc != HILBERTA_OK) {
        free_plan(p);
        return rc;
    }
    *out = p;
    return HILBERTA_OK;
}

extern "C" int hilberta_plan(int H, int W, int tile, int layer_offset, int shared_region, int n_text,
                             hilberta_plan_t **out) {
    if (tile < 1) {
        if (out) *out = nullptr;
        return HILBERTA_ERR_INVALID;
    }
    return make_plan(1, H, W, tile, 0, layer_offset, shared_region, 0, n_text, out);
}

extern "C" int hilberta_plan_groups(int H, int W, int groups, int layer_offset, int shared_region, int n_text,
                                    hilberta_plan_t **out) {
    if (groups < 1) {
        if (out) *out = nullptr;
        return HILBERTA_ERR_INVALID;
    }
    return make_plan(1, H, W, 0, groups, layer_offset, shared_region, 0, n_text, out);
}

extern "C" int hilberta_plan_video(int frames, int H, int W, int tile, int layer_offset, int shared_region,
                                   int shared_frames, int n_text, hilberta_plan_t **out) {
    if (tile < 1 || frames < 2) {
        if (out) *out = nullptr;
        return HILBERTA_ERR_INVALID;
    }
    return make_plan(frames, H, W, tile, 0, layer_offset, shared_region, shared_frames, n_text, out);
}

extern "C" int hilberta_plan_destroy(hilberta_plan_t *plan) {
    free_plan(plan);
    return HILBERTA_OK;
}

extern "C" int hilberta_plan_export(const hilberta_plan_t *p, int what, void *host_buf, size_t bytes,
                                    size_t *needed) {
    if (!p) return HILBERTA_ERR_INVALID;
    size_t need = 0;
    const void *dsrc = nullptr;
    std::vector<int> tmp;
    uint64_t nnz = p->nnz;
    const void *hsrc = nullptr;
    switch (what) {
        case HILBERTA_EXPORT_HIL_D2T: need = sizeof(int) * p->HW; dsrc = p->d_hil_d2t; break;
        case HILBERTA_EXPORT_HIL_T2D: need = sizeof(int) * p->HW; dsrc = p->d_hil_t2d; break;
        case HILBERTA_EXPORT_PHYS2ORIG: need = sizeof(int) * p->S; dsrc = p->d_phys2orig; break;
        case HILBERTA_EXPORT_ORIG2PHYS: need = sizeof(int) * p->S; dsrc = p->d_orig2phys; break;
        case HILBERTA_EXPORT_SHARED_RUNS:
            need = sizeof(int) * p->h_shared_runs.size();
            hsrc = p->h_shared_runs.data();
            break;
        case HILBERTA_EXPORT_WINDOWS:
            need = sizeof(Window) * p->h_windows.size();
            hsrc = p->h_windows.data();
            break;
        case HILBERTA_EXPORT_NNZ: need = sizeof(uint64_t); hsrc = &nnz; break;
        case HILBERTA_EXPORT_INFO:
            tmp = {p->H, p->W, p->tile, p->offset, p->shared_region, p->n_text, p->n_shared, p->T, 1 << p->k_log2,
                   p->frames, p->shared_frames};
            need = sizeof(int) * tmp.size();
            hsrc = tmp.data();
            break;
        case HILBERTA_EXPORT_LAUNCH_CLOCK:
            need = sizeof(int) * 2;
            dsrc = p->d_status + 32;
            if (host_buf) HB_CUDA(cudaDeviceSynchronize());
            break;
#if defined(HB_TIMING) || defined(HB_STAMPS)
        case 100: need = sizeof(int) * 4096; dsrc = p->d_status; break;  // role cycle counters and event trace
#endif
        default: return HILBERTA_ERR_INVALID;
    }
    if (needed) *needed = need;
    if (!host_buf) return HILBERTA_OK;
    if (bytes < need) return HILBERTA_ERR_BUFFER;
    if (dsrc) {
        HB_CUDA(cudaMemcpy(host_buf, dsrc, need, cudaMemcpyDeviceToHost));
    } else if (need) {
        memcpy(host_buf, hsrc, need);
    }
    return HILBERTA_OK;
}

extern "C" int hilberta_plan_bind(hilberta_plan_t *p, int batch, int heads, int head_dim, int dtype,
                                  int64_t stride_b, int64_t stride_h, int64_t stride_s, float scale) {
    if (!p || batch < 1 || heads < 1 || head_dim < 1) return HILBERTA_ERR_INVALID;
    if (dtype != HILBERTA_BF16 && dtype != HILBERTA_FP32 && dtype != HILBERTA_FP8_E4M3) return HILBERTA_ERR_INVALID;
    if (dtype == HILBERTA_BF16 && head_dim != 128 && head_dim != 64) return HILBERTA_ERR_UNSUPPORTED;
    if (dtype == HILBERTA_FP8_E4M3 && head_dim != 128) return HILBERTA_ERR_UNSUPPORTED;
    if (dtype == HILBERTA_FP32 && head_dim != 32 && head_dim != 64 && head_dim != 128)
        return HILBERTA_ERR_UNSUPPORTED;
    if (stride_b == 0 && stride_h == 0 && stride_s == 0) {
        stride_s = head_dim;
        stride_h = (int64_t)p->S * head_dim;
        stride_b = (int64_t)heads * stride_h;
    }
    if (stride_b <= 0 || stride_h <= 0 || stride_s < head_dim) return HILBERTA_ERR_INVALID;
    if (dtype == HILBERTA_BF16 && ((stride_b | stride_h | stride_s) & 7)) return HILBERTA_ERR_INVALID;
    if (dtype == HILBERTA_FP8_E4M3 && ((stride_b | stride_h | stride_s) & 15)) return HILBERTA_ERR_INVALID;
    if ((int64_t)batch * heads > 65535) return HILBERTA_ERR_INVALID;
    p->bound = false;
    p->batch = batch;
    p->heads = heads;
    p->head_dim = head_dim;
    p->dtype = dtype;
    p->stride_b = stride_b;
    p->stride_h = stride_h;
    p->stride_s = stride_s;
    p->scale = scale > 0.f ? scale : 1.0f / sqrtf((float)head_dim);
    if (dtype == HILBERTA_BF16) {
        int rc = attn_bf16_prepare(p);
        if (rc != HILBERTA_OK) return rc;
        rc = attn_bwd_prepare(p);
        if (rc != HILBERTA_OK) return rc;
    }
    if (dtype == HILBERTA_FP8_E4M3) {
        // forward only: the bf16 kernel's work list and schedule, no backward tables
        int rc = attn_bf16_prepare(p);
        if (rc != HILBERTA_OK) return rc;
    }
    if (dtype == HILBERTA_FP32) {
        // scratch of the backward pass (delta per row; sized like the bf16 path's)
        cudaFree(p->d_delta);
        p->d_delta = nullptr;
        HB_CUDA(cudaMalloc(&p->d_delta, sizeof(float) * 2 * (size_t)batch * heads * p->S));
    }
    p->bound = true;
    return HILBERTA_OK;
}

// Do two tensors of the layout [batch, heads, S, row] share a byte?  Both use the byte strides sb, sh,
// ss and rows of row_bytes contiguous bytes; a and b are their base addresses.  Exact: the tensors
// overlap iff b - a = dx sb + dy sh + dz ss + dc for some |dx| < batch, |dy| < heads, |dz| < S,
// |dc| < row_bytes (every such difference of indices is the difference of two valid indices).  So
// tensors interleaved in one buffer (q, k, v and out as slices of one packed array) pass, and any
// real overlap -- a shifted copy of an input used as output -- is caught.
static bool layouts_overlap(uint64_t a, uint64_t b, int batch, int heads, int S, int64_t sb, int64_t sh, int64_t ss,
                            int64_t row_bytes) {
    if (batch < 1 || heads < 1 || S < 1 || row_bytes < 1) return false;
    const int64_t d = (int64_t)(b - a);
    if (ss <= 0) {
        // no usable token stride: compare the address ranges
        const int64_t ext = (batch - 1) * llabs(sb) + (heads - 1) * llabs(sh) + (int64_t)(S - 1) * llabs(ss) + row_bytes;
        return d < ext && -d < ext;
    }
    for (int dx = -(batch - 1); dx <= batch - 1; ++dx)
        for (int dy = -(heads - 1); dy <= heads - 1; ++dy) {
            const int64_t rem = d - dx * sb - dy * sh;
            int64_t dz = rem / ss;   // rem = dz ss + dc: dz is the quotient rounded toward zero or its neighbours
            for (int64_t z = dz - 1; z <= dz + 1; ++z)
                if (z > -(int64_t)S && z < (int64_t)S && llabs(rem - z * ss) < row_bytes) return true;
        }
    return false;
}

extern "C" int hilberta_check_overlap(uint64_t a, uint64_t b, int batch, int heads, int S, int64_t stride_b_bytes,
                                      int64_t stride_h_bytes, int64_t stride_s_bytes, int64_t row_bytes) {
    return layouts_overlap(a, b, batch, heads, S, stride_b_bytes, stride_h_bytes, stride_s_bytes, row_bytes) ? 1 : 0;
}

namespace hilberta {
// `out` (element size esz_out) against `in` (element size esz_in) on the plan's bound layout.  Equal
// element sizes: the exact test.  e4m3 inputs with a bf16 output use different byte strides: there
// the address ranges are compared.
bool bound_tensors_overlap(const hilberta_plan_t *p, const void *out, size_t esz_out, const void *in, size_t esz_in) {
    const uint64_t a = (uint64_t)(uintptr_t)out, b = (uint64_t)(uintptr_t)in;
    if (esz_out == esz_in)
        return layouts_overlap(a, b, p->batch, p->heads, p->S, p->stride_b * (int64_t)esz_out, p->stride_h * (int64_t)esz_out,
                               p->stride_s * (int64_t)esz_out, (int64_t)p->head_dim * (int64_t)esz_out);
    auto extent = [&](size_t esz) {
        return (uint64_t)(((int64_t)(p->batch - 1) * p->stride_b + (int64_t)(p->heads - 1) * p->stride_h +
                           (int64_t)(p->S - 1) * p->stride_s + p->head_dim) * (int64_t)esz);
    };
    return a < b + extent(esz_in) && b < a + extent(esz_out);
}
}  // namespace hilberta

static int forward_impl(const void *q, const void *k, const void *v, void *out, float *lse,
                        const hilberta_plan_t *p, const int *out_map, const int *in_map, void *stream,
                        int chunk = -1) {
    if (!p || !q || !k || !v || !out) return HILBERTA_ERR_INVALID;
    if (!p->bound) return HILBERTA_ERR_UNBOUND;
    {
        // `out` must not share a byte with an input (other launches' reads would race with its writes)
        const size_t esz_in = p->dtype == HILBERTA_BF16 ? 2 : p->dtype == HILBERTA_FP8_E4M3 ? 1 : 4;
        const size_t esz_out = p->dtype == HILBERTA_FP8_E4M3 ? 2 : esz_in;
        const void *in[3] = {q, k, v};
        for (int i = 0; i < 3; ++i)
            if (hilberta::bound_tensors_overlap(p, out, esz_out, in[i], esz_in)) return HILBERTA_ERR_INVALID;
    }
    int dev = -1;
    HB_CUDA(cudaGetDevice(&dev));
    if (dev != p->device) return HILBERTA_ERR_INVALID;  // the plan's tables live on another device
    cudaStream_t st = (cudaStream_t)stream;
    if (p->dtype == HILBERTA_FP32) return launch_attn_fp32(p, q, k, v, out, lse, out_map, in_map, st, chunk);
    const uintptr_t bits = (uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out;
    if (bits & 15) return HILBERTA_ERR_INVALID;
    return launch_attn_bf16(p, q, k, v, out, lse, out_map, in_map, st, chunk);
}

extern "C" int hilberta_forward(const void *q, const void *k, const void *v, void *out,
                                const hilberta_plan_t *p, void *stream) {
    return forward_impl(q, k, v, out, nullptr, p, nullptr, nullptr, stream);
}

extern "C" int hilberta_forward_unpermute(const void *q, const void *k, const void *v, void *out,
                                          const hilberta_plan_t *p, void *stream) {
    return forward_impl(q, k, v, out, nullptr, p, p ? p->d_phys2orig : nullptr, nullptr, stream);
}

extern "C" int hilberta_forward_fused(const void *q, const void *k, const void *v, void *out,
                                      const hilberta_plan_t *p, int in_original, int out_original, void *stream) {
    const int *map = p ? p->d_phys2orig : nullptr;
    return forward_impl(q, k, v, out, nullptr, p, out_original ? map : nullptr, in_original ? map : nullptr, stream);
}

extern "C" int hilberta_forward_lse(const void *q, const void *k, const void *v, void *out, float *lse,
                                    const hilberta_plan_t *p, void *stream) {
    if (!lse || ((uintptr_t)lse & 3)) return HILBERTA_ERR_INVALID;
    return forward_impl(q, k, v, out, lse, p, nullptr, nullptr, stream);
}

extern "C" int hilberta_backward(const void *dout, const void *q, const void *k, const void *v, const void *out,
                                 const float *lse, void *dq, void *dk, void *dv, const hilberta_plan_t *p,
                                 void *stream) {
    if (!p || !dout || !q || !k || !v || !out || !lse || !dq || !dk || !dv) return HILBERTA_ERR_INVALID;
    if (!p->bound) return HILBERTA_ERR_UNBOUND;
    const void *in[5] = {dout, q, k, v, out};
    void *outs[3] = {dq, dk, dv};
    uintptr_t bits = (uintptr_t)lse & 3 ? 15 : 0;
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
    return launch_attn_bwd(p, dout, q, k, v, out, lse, dq, dk, dv, p->d_delta, (cudaStream_t)stream);
}

// Whole path for host-resident activations.  The heads are processed in slices: the H2D copies of
// slice c + 1 (own stream), the ONE launch of slice c (reads q, k, v through the permutation and
// writes `out` in the original order: entry and exit gathers fused in) and the D2H copy of slice
// c - 1 (own stream) overlap, so the two PCIe directions work at the same time.  Four device
// buffers of one tensor each.
extern "C" int hilberta_forward_host(const void *q, const void *k, const void *v, void *out,
                                     hilberta_plan_t *p, void *stream) {
    if (!p || !q || !k || !v || !out) return HILBERTA_ERR_INVALID;
    if (!p->bound) return HILBERTA_ERR_UNBOUND;
    const int64_t dense_h = (int64_t)p->S * p->head_dim;
    if (p->stride_s != p->head_dim || p->stride_h != dense_h || p->stride_b != dense_h * p->heads)
        return HILBERTA_ERR_INVALID;
    int dev = -1;
    HB_CUDA(cudaGetDevice(&dev));
    if (dev != p->device) return HILBERTA_ERR_INVALID;
    // element sizes of q, k, v and of out (e4m3 bindings: 8-bit inputs, bf16 output)
    const size_t esz = p->dtype == HILBERTA_BF16 ? 2 : p->dtype == HILBERTA_FP8_E4M3 ? 1 : 4;
    const size_t esz_out = p->dtype == HILBERTA_FP8_E4M3 ? 2 : esz;
    const size_t bytes = (size_t)p->batch * p->heads * p->S * p->head_dim * esz_out;   // the larger of the two
    const size_t slot = (bytes + 255) & ~(size_t)255;
    if (p->ws_bytes < 4 * slot) {
        cudaFree(p->ws);
        p->ws = nullptr;
        p->ws_bytes = 0;
        HB_CUDA(cudaMalloc(&p->ws, 4 * slot));
        p->ws_bytes = 4 * slot;
    }
    // fp32 bindings have no slice schedule to build: chunk_heads is only set by the bf16 path
    const int hc = (p->dtype != HILBERTA_FP32 && p->chunk_heads > 0) ? p->chunk_heads : p->heads;
    const int n_chunks = p->heads / hc;
    if (!p->s_in) HB_CUDA(cudaStreamCreateWithFlags(&p->s_in, cudaStreamNonBlocking));
    if (!p->s_out) HB_CUDA(cudaStreamCreateWithFlags(&p->s_out, cudaStreamNonBlocking));
    while ((int)p->ev_in.size() < n_chunks + 1) {
        cudaEvent_t e0, e1;
        HB_CUDA(cudaEventCreateWithFlags(&e0, cudaEventDisableTiming));
        HB_CUDA(cudaEventCreateWithFlags(&e1, cudaEventDisableTiming));
        p->ev_in.push_back(e0);
        p->ev_done.push_back(e1);
    }
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = (char *)p->ws;
    void *in[3] = {ws, ws + slot, ws + 2 * slot};
    char *out_dev = ws + 3 * slot;
    const void *host_in[3] = {q, k, v};
    // a slice of hc heads of every batch item: `batch` rows of row_bytes, one tensor of heads apart
    const size_t row_bytes = (size_t)hc * p->S * p->head_dim * esz;
    const size_t pitch = (size_t)p->heads * p->S * p->head_dim * esz;
    const size_t row_bytes_out = row_bytes / esz * esz_out, pitch_out = pitch / esz * esz_out;
    // work already queued on the caller's stream comes first
    HB_CUDA(cudaEventRecord(p->ev_in[n_chunks], st));
    HB_CUDA(cudaStreamWaitEvent(p->s_in, p->ev_in[n_chunks], 0));
    for (int c = 0; c < n_chunks; ++c) {
        const size_t off = (size_t)c * row_bytes;
        for (int i = 0; i < 3; ++i)
            HB_CUDA(cudaMemcpy2DAsync((char *)in[i] + off, pitch, (const char *)host_in[i] + off, pitch, row_bytes,
                                      p->batch, cudaMemcpyHostToDevice, p->s_in));
        HB_CUDA(cudaEventRecord(p->ev_in[c], p->s_in));
        HB_CUDA(cudaStreamWaitEvent(st, p->ev_in[c], 0));
        const int rc = forward_impl(in[0], in[1], in[2], out_dev, nullptr, p, p->d_phys2orig, p->d_phys2orig, st,
                                    n_chunks > 1 ? c : -1);
        if (rc != HILBERTA_OK) return rc;
        HB_CUDA(cudaEventRecord(p->ev_done[c], st));
        HB_CUDA(cudaStreamWaitEvent(p->s_out, p->ev_done[c], 0));
        const size_t off_out = (size_t)c * row_bytes_out;
        HB_CUDA(cudaMemcpy2DAsync((char *)out + off_out, pitch_out, out_dev + off_out, pitch_out, row_bytes_out, p->batch,
                                  cudaMemcpyDeviceToHost, p->s_out));
    }
    HB_CUDA(cudaStreamSynchronize(p->s_out));
    HB_CUDA(cudaStreamSynchronize(st));
    return HILBERTA_OK;
}

extern "C" int hilberta_selftest_timeout(hilberta_plan_t *p, void *stream) {
    if (!p) return HILBERTA_ERR_INVALID;
    return launch_timeout_probe(p, (cudaStream_t)stream);
}

extern "C" int hilberta_plan_status(hilberta_plan_t *p) {
    if (!p) return HILBERTA_ERR_INVALID;
    int h[4] = {0, 0, 0, 0};
    HB_CUDA(cudaDeviceSynchronize());
    HB_CUDA(cudaMemcpy(h, p->d_status, sizeof(h), cudaMemcpyDeviceToHost));
    if (h[0] != 0) {
        HB_CUDA(cudaMemset(p->d_status, 0, sizeof(h)));
        return HILBERTA_ERR_TIMEOUT;
    }
    return HILBERTA_OK;
}

extern "C" uint64_t hilberta_launch_count(void) { return g_launches.load(); }

extern "C" const char *hilberta_status_string(int status) {
    switch (status) {
        case HILBERTA_OK: return "ok";
        case HILBERTA_ERR_INVALID: return "invalid argument";
        case HILBERTA_ERR_UNSUPPORTED: return "unsupported shape";
        case HILBERTA_ERR_ARCH: return "device is not sm_100";
        case HILBERTA_ERR_CUDA: return "CUDA error";
        case HILBERTA_ERR_NOMEM: return "out of memory";
        case HILBERTA_ERR_BUFFER: return "buffer too small";
        case HILBERTA_ERR_UNBOUND: return "plan not bound to a problem shape";
        case HILBERTA_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

extern "C" int hilberta_version(void) { return HILBERTA_VERSION; }

extern "C" int hilberta_last_cuda_error(void) { return g_last_cuda_error; }
