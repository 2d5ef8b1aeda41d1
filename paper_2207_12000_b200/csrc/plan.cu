// Plan construction: degrees, operator scales, the support's edge list, the balanced edge blocks
// (Section 3.2, "Precomputation on GPU"; Algorithm 1's split of S), Eq. 12's block counts, and the
// warp-level segment tables the propagation kernels walk.  All of it runs on the GPU except the
// O(b) block arithmetic and the Eq. 12 search.
#include <algorithm>
#include <cstring>
#include <new>

#include "gnnpre_internal.cuh"

namespace gnnpre {

namespace {

constexpr int kTB = 256;

inline unsigned grid_for(int64_t items, int per_block) {
    int64_t g = (items + per_block - 1) / per_block;
    return (unsigned)std::max<int64_t>(1, g);
}

// ---------------------------------------------------------------- validation, degrees, scales

enum : int { kErrRowptr = 1, kErrColRange = 2, kErrDiagonal = 4, kErrOrder = 8, kErrDegree = 16 };

// One warp per row: checks the input contract of the CSR.
__global__ void k_validate(int64_t n, int64_t nnz, const int64_t* __restrict__ rowptr,
                           const int32_t* __restrict__ colidx, int* err) {
    const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= n) return;
    const int64_t lo = rowptr[row], hi = rowptr[row + 1];
    int bad = 0;
    if (lo < 0 || hi < lo || hi > nnz) {
        bad |= kErrRowptr;
    } else {
        if (hi - lo >= 0x7fffffffLL) bad |= kErrDegree;
        for (int64_t e = lo + lane; e < hi; e += 32) {
            const int32_t c = colidx[e];
            if (c < 0 || c >= n) bad |= kErrColRange;
            if (c == row) bad |= kErrDiagonal;
            if (e + 1 < hi && colidx[e + 1] <= c) bad |= kErrOrder;
        }
    }
    if (bad) atomicOr(err, bad);
}

// D_i = number of nonzeros in row i of A (Section 2).
__global__ void k_degrees(int64_t n, const int64_t* __restrict__ rowptr, int32_t* __restrict__ deg) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) deg[i] = (int32_t)(rowptr[i + 1] - rowptr[i]);
}

// A^_ij = r_i c_j: GCN r = c = (D_i + 1)^{-1/2} (Eq. 1); SAGE r = 1/D_i (0 for D_i = 0), c = 1;
// GIN r = c = 1.  Evaluated in fp64 (IEEE sqrt and divide) and rounded once to fp32.
__global__ void k_scales(int op, int64_t n, const int32_t* __restrict__ deg, float* __restrict__ rscale,
                         float* __restrict__ cscale) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    double r = 1.0, c = 1.0;
    if (op == GNNPRE_OP_GCN_SYM) {
        r = c = 1.0 / sqrt((double)deg[i] + 1.0);
    } else if (op == GNNPRE_OP_SAGE_MEAN) {
        r = deg[i] > 0 ? 1.0 / (double)deg[i] : 0.0;
    }
    rscale[i] = (float)r;
    cscale[i] = (float)c;
}

// ---------------------------------------------------------------- the support's edge list E

// One warp per row.  With `diag`, row i of the support is row i of A plus the self-loop (i, i) at
// its column-sorted position, so rowptr_t[i] = rowptr[i] + i.  The last entry of every non-empty
// row carries kRowEndBit.
__global__ void k_support(int diag, int64_t n, const int64_t* __restrict__ rowptr, const int32_t* __restrict__ colidx,
                          int64_t* __restrict__ rowptr_t, uint32_t* __restrict__ colx) {
    const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= n) return;
    const int64_t lo = rowptr[row], hi = rowptr[row + 1];
    const int64_t base = lo + (diag ? row : 0);
    const int64_t len_t = hi - lo + (diag ? 1 : 0);
    if (lane == 0) {
        rowptr_t[row] = base;
        if (row == n - 1) rowptr_t[n] = base + len_t;
    }
    int64_t below = 0;  // entries of the row with column < row
    for (int64_t e0 = lo; e0 < hi; e0 += 32) {
        const int64_t e = e0 + lane;
        bool lt = false;
        if (e < hi) {
            const int32_t c = colidx[e];
            lt = c < row;
            const int64_t pos = (e - lo) + ((diag && !lt) ? 1 : 0);
            colx[base + pos] = (uint32_t)c | (pos == len_t - 1 ? kRowEndBit : 0u);
        }
        below += __popc(__ballot_sync(0xffffffffu, lt));
    }
    if (diag && lane == 0) colx[base + below] = (uint32_t)row | (below == len_t - 1 ? kRowEndBit : 0u);
}

// ---------------------------------------------------------------- exclusive scan (int32)

constexpr int kScanItems = 8;
constexpr int kScanTile = kTB * kScanItems;

__device__ __forceinline__ int block_exclusive_scan(int v, int* total) {
    __shared__ int warp_sums[kTB / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += t;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = lane < kTB / 32 ? warp_sums[lane] : 0;
#pragma unroll
        for (int d = 1; d < kTB / 32; d <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, w, d);
            if (lane >= d) w += t;
        }
        if (lane < kTB / 32) warp_sums[lane] = w;  // inclusive over warps
    }
    __syncthreads();
    const int warp_off = warp > 0 ? warp_sums[warp - 1] : 0;
    *total = warp_sums[kTB / 32 - 1];
    const int r = warp_off + incl - v;
    __syncthreads();
    return r;
}

__global__ void k_tile_sums(const int32_t* __restrict__ in, int64_t n, int32_t* __restrict__ sums) {
    const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
    int s = 0;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k)
        if (base + k < n) s += in[base + k];
    int total;
    block_exclusive_scan(s, &total);
    if (threadIdx.x == 0) sums[blockIdx.x] = total;
}

// out[i] = tile_off[tile] + exclusive prefix inside the tile; the last tile also writes out[n] = grand total.
__global__ void k_tile_scan(const int32_t* __restrict__ in, int64_t n, const int32_t* __restrict__ tile_off,
                            int32_t* __restrict__ out) {
    const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
    int v[kScanItems];
    int s = 0;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
        v[k] = base + k < n ? in[base + k] : 0;
        s += v[k];
    }
    int total;
    int run = block_exclusive_scan(s, &total) + (tile_off ? tile_off[blockIdx.x] : 0);
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
        if (base + k < n) out[base + k] = run;
        run += v[k];
        if (base + k == n - 1) out[n] = run;
    }
}

// out has n + 1 entries: exclusive prefix sums and the total.  `in` and `out` may not alias.
int exclusive_scan(const int32_t* in, int64_t n, int32_t* out, cudaStream_t st) {
    if (n == 0) {
        GNNPRE_CUDA(cudaMemsetAsync(out, 0, sizeof(int32_t), st));
        return GNNPRE_OK;
    }
    const int64_t tiles = (n + kScanTile - 1) / kScanTile;
    if (tiles == 1) {
        k_tile_scan<<<1, kTB, 0, st>>>(in, n, nullptr, out);
        GNNPRE_CUDA(cudaGetLastError());
        return GNNPRE_OK;
    }
    DevBuf<int32_t> sums, offs;
    GNNPRE_TRY(sums.alloc((size_t)tiles));
    GNNPRE_TRY(offs.alloc((size_t)tiles + 1));
    k_tile_sums<<<(unsigned)tiles, kTB, 0, st>>>(in, n, sums.p);
    GNNPRE_CUDA(cudaGetLastError());
    GNNPRE_TRY(exclusive_scan(sums.p, tiles, offs.p, st));
    k_tile_scan<<<(unsigned)tiles, kTB, 0, st>>>(in, n, offs.p, out);
    GNNPRE_CUDA(cudaGetLastError());
    GNNPRE_CUDA(cudaStreamSynchronize(st));  // temporaries die here
    return GNNPRE_OK;
}

// ---------------------------------------------------------------- rows of edges

// Row holding edge e of the support: the last i with rowptr_t[i] <= e (rows without edges are skipped
// because their successor shares their start).
__device__ __forceinline__ int64_t row_of_edge(const int64_t* __restrict__ rowptr_t, int64_t n, int64_t e) {
    int64_t lo = 0, hi = n;  // invariant: rowptr_t[lo] <= e < rowptr_t[hi]
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (rowptr_t[mid] <= e) lo = mid; else hi = mid;
    }
    return lo;
}

struct BlockRows {
    int32_t row_lo, row_hi, first_partial, last_partial;
    int64_t done_row_hi;
};

__global__ void k_block_rows(int b, const int64_t* __restrict__ e_off, const int64_t* __restrict__ rowptr_t,
                             int64_t n, BlockRows* __restrict__ out) {
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l >= b) return;
    const int64_t lo = e_off[l], hi = e_off[l + 1];
    const int64_t r0 = row_of_edge(rowptr_t, n, lo), r1 = row_of_edge(rowptr_t, n, hi - 1);
    BlockRows o;
    o.row_lo = (int32_t)r0;
    o.row_hi = (int32_t)r1;
    o.first_partial = rowptr_t[r0] < lo;
    o.last_partial = rowptr_t[r1 + 1] > hi;
    // rows complete after this block: every row whose end offset is <= hi
    int64_t a = 0, z = n;  // count of i in [0, n) with rowptr_t[i + 1] <= hi
    while (a < z) {
        const int64_t mid = (a + z) >> 1;
        if (rowptr_t[mid + 1] <= hi) a = mid + 1; else z = mid;
    }
    o.done_row_hi = a;
    out[l] = o;
}

// ---------------------------------------------------------------- rows with and without edges

__global__ void k_nonempty_flags(int64_t n, const int64_t* __restrict__ rowptr_t, int32_t* __restrict__ flag) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) flag[i] = rowptr_t[i + 1] > rowptr_t[i];
}

__global__ void k_split_rows(int64_t n, const int32_t* __restrict__ flag, const int32_t* __restrict__ rank,
                             int32_t* __restrict__ nzrows, int32_t* __restrict__ emptyrows) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    if (flag[i]) nzrows[rank[i]] = (int32_t)i; else emptyrows[i - rank[i]] = (int32_t)i;
}

// ---------------------------------------------------------------- warp-level segments

// Segment t of block l nominally starts at e_lo(l) + t*L.  A start that falls inside a row is moved
// forward to the next row start when that lies within `snap` edges (and inside the block), so that
// short rows are never cut; long rows are cut and their parts summed by a fix-up.
// Temporarily: slot_head holds the "first row began earlier" flag and pad holds the first row's index.
__global__ void k_segment_starts(int64_t nseg, int b, const int64_t* __restrict__ seg_base,
                                 const int64_t* __restrict__ e_off, int32_t L, int32_t snap,
                                 const int64_t* __restrict__ rowptr_t, int64_t n, const int32_t* __restrict__ rank,
                                 Segment* __restrict__ segs) {
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s > nseg) return;
    Segment g;
    if (s == nseg) {  // sentinel
        g.start = e_off[b];
        g.rank = 0;
        g.slot_head = 0;
        g.slot_tail = -1;
        g.pad = (int32_t)n;
        segs[s] = g;
        return;
    }
    int lo = 0, hi = b;  // block holding segment s: seg_base[lo] <= s < seg_base[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (seg_base[mid] <= s) lo = mid; else hi = mid;
    }
    const int64_t t = s - seg_base[lo];
    int64_t start = e_off[lo] + t * (int64_t)L;
    int64_t row = row_of_edge(rowptr_t, n, start);
    if (t > 0 && rowptr_t[row] < start) {
        const int64_t next = rowptr_t[row + 1];
        if (next - start <= snap && next < e_off[lo + 1]) {
            start = next;
            row = row_of_edge(rowptr_t, n, start);
        }
    }
    g.start = start;
    g.rank = rank ? rank[row] : (int32_t)row;
    g.slot_head = rowptr_t[row] < start;
    g.slot_tail = -1;
    g.pad = (int32_t)row;
    segs[s] = g;
}

// flags[2s] = segment s needs a head slot; flags[2s+1] = it needs a tail slot; emit[s] = the row
// that began before segment s ends inside it (one fix-up per such row).
__global__ void k_segment_flags(int64_t nseg, const Segment* __restrict__ segs, const int64_t* __restrict__ rowptr_t,
                                int32_t* __restrict__ flags, int32_t* __restrict__ emit) {
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= nseg) return;
    const Segment g = segs[s], nx = segs[s + 1];
    const int head = g.slot_head;
    // the row holding this segment's last edge continues iff the next segment's first row began earlier
    const int tail = nx.slot_head && rowptr_t[nx.pad] >= g.start;
    flags[2 * s] = head;
    flags[2 * s + 1] = tail;
    emit[s] = head && rowptr_t[(int64_t)g.pad + 1] <= nx.start;
}

__global__ void k_segment_finalize(int64_t nseg, Segment* __restrict__ segs, const int64_t* __restrict__ rowptr_t,
                                   const int32_t* __restrict__ flags, const int32_t* __restrict__ slot_scan,
                                   const int32_t* __restrict__ emit, const int32_t* __restrict__ emit_scan,
                                   RowFixup* __restrict__ fixups) {
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= nseg) return;
    const int32_t row = segs[s].pad;
    if (emit[s]) {
        const int64_t first_edge = rowptr_t[row];
        int64_t lo = 0, hi = s;  // segs[lo].start <= first_edge < segs[hi].start
        while (hi - lo > 1) {
            const int64_t mid = (lo + hi) >> 1;
            if (segs[mid].start <= first_edge) lo = mid; else hi = mid;
        }
        RowFixup f;
        f.row = row;
        f.seg_first = (int32_t)lo;
        f.seg_last = (int32_t)s;
        f.slot0 = slot_scan[2 * lo + 1];  // the tail slot of the row's first segment; the other parts follow it
        fixups[emit_scan[s]] = f;
    }
    segs[s].slot_head = flags[2 * s] ? slot_scan[2 * s] : -1;
    segs[s].slot_tail = flags[2 * s + 1] ? slot_scan[2 * s + 1] : -1;
}

__global__ void k_hub_flags(int64_t nfix, const RowFixup* __restrict__ fix, int32_t hub_parts, int32_t* __restrict__ flag) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < nfix) flag[i] = fix[i].seg_last - fix[i].seg_first + 1 > hub_parts;
}

__global__ void k_hub_scatter(int64_t nfix, const int32_t* __restrict__ flag, const int32_t* __restrict__ scan,
                              int32_t* __restrict__ hubs) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < nfix && flag[i]) hubs[scan[i]] = (int32_t)i;
}

// Parts beyond which a cut row counts as a hub and gets a whole CTA of the fix-up kernel (64 chains) instead of a
// warp (8 chains).  One value for all widths up to 128 columns, because the tree's shape decides the bits and
// those must not depend on how a matrix is cut into column tiles; wider tiles hold fewer parts per batch of loads.
int32_t hub_parts_for(int64_t width) {
    const int64_t f4 = std::min<int64_t>(std::max<int64_t>(width, 4), 512) / 4;
    return f4 <= 32 ? 64 : f4 <= 64 ? 32 : 16;
}

__global__ void k_clear_pad(int64_t nseg, Segment* __restrict__ segs) {
    const int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s <= nseg) segs[s].pad = 0;
}

__global__ void k_gather_i32(int count, const int64_t* __restrict__ idx, const int32_t* __restrict__ src,
                             int32_t* __restrict__ dst) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) dst[i] = src[idx[i]];
}

int32_t auto_segment_edges(int64_t slab_width, int64_t m, bool bulk_copy, int num_sms) {
    if (bulk_copy) {
        // persistent warps walk whole segments with a two-stage pipeline that drains at every segment
        // end: long segments, but at least ~4 per resident warp so the tail stays short
        const int64_t per_warp = m / ((int64_t)std::max(num_sms, 1) * 16 * 4);
        int32_t p = 256;
        while ((int64_t)p * 2 <= per_warp && p < 4096) p *= 2;
        return p;
    }
    // about 32 Ki gathered floats per segment, but short enough that every SM's 2048 threads get a
    // segment per lane group; a power of two between 32 and 4096 edges.  Rows wider than 256 floats
    // get at least 128 edges per segment (256 when the graph still leaves a thousand edges per lane
    // group): with shorter ones most rows are cut and adding up their parts costs more than the
    // segments save (F = 602, 23 M edges: 17.0 ms per two hops at 32 edges, 13.5 ms at 256).
    const int64_t f4 = std::min<int64_t>(std::max<int64_t>(slab_width, 4), 512) / 4;
    const int64_t lanes = f4 <= 4 ? 4 : f4 <= 8 ? 8 : f4 <= 16 ? 16 : 32;
    const int64_t groups = (int64_t)std::max(num_sms, 1) * (2048 / lanes);
    int64_t by_width = 32768 / std::max<int64_t>(slab_width, 4);
    if (by_width < 128) by_width = m / groups >= 1024 ? 256 : 128;
    const int64_t L = std::min<int64_t>(by_width, m / groups);
    int32_t p = 32;
    while ((int64_t)p * 2 <= L && p < 4096) p *= 2;
    return p;
}

}  // namespace

// ---------------------------------------------------------------- Eq. 12

// For a fixed c the least feasible b has a closed form, so one pass over c suffices.
int solve_budget(int64_t B_S, int64_t B_X, int64_t B_fixed, int64_t beta_S, int64_t beta_X, int64_t B_GPU,
                 int64_t max_b, int64_t max_c, int64_t* b_out, int64_t* c_out) {
    if (B_S < 0 || B_X < 0 || B_fixed < 0 || beta_S < 1 || beta_X < 1 || max_b < 1 || max_c < 1)
        return GNNPRE_ERR_INVALID_ARG;
    bool found = false;
    int64_t best_b = 0, best_c = 0;
    const int64_t need_S = beta_S * B_S;
    for (int64_t c = 1; c <= max_c; ++c) {
        const int64_t x_part = (beta_X * B_X + c - 1) / c;
        const int64_t room = B_GPU - B_fixed - x_part;
        if (room <= 0 && need_S > 0) continue;
        if (room < 0) continue;
        const int64_t b = need_S == 0 ? 1 : (need_S + room - 1) / room;
        if (b > max_b) continue;
        const int64_t bb = std::max<int64_t>(b, 1);
        if (!found || bb * c < best_b * best_c) {  // ascending c: the first minimum has the smallest c
            found = true;
            best_b = bb;
            best_c = c;
        }
    }
    if (!found) return GNNPRE_ERR_BUDGET_TOO_SMALL;
    *b_out = best_b;
    *c_out = best_c;
    return GNNPRE_OK;
}

int check_device_error(gnnpre_plan* P) {
    if (!P->dev_error.p) return GNNPRE_OK;
    int h = 0;
    GNNPRE_CUDA(cudaMemcpy(&h, P->dev_error.p, sizeof(int), cudaMemcpyDeviceToHost));
    if (h == 0) return GNNPRE_OK;
    GNNPRE_CUDA(cudaMemset(P->dev_error.p, 0, sizeof(int)));
    return GNNPRE_ERR_TIMEOUT;
}

int check_device() {
    int dev = 0;
    GNNPRE_CUDA(cudaGetDevice(&dev));
    int major = 0;
    GNNPRE_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    return major == 10 ? GNNPRE_OK : GNNPRE_ERR_UNSUPPORTED_ARCH;
}

}  // namespace gnnpre

using namespace gnnpre;

gnnpre_plan::~gnnpre_plan() {
    if (s_h2d) cudaStreamDestroy(s_h2d);
    if (s_d2h) cudaStreamDestroy(s_d2h);
    if (s_compute) cudaStreamDestroy(s_compute);
    if (s_struct) cudaStreamDestroy(s_struct);
    if (last_use) cudaEventDestroy(last_use);
}

int64_t gnnpre_plan::device_bytes() const {
    size_t t = deg.bytes() + rscale.bytes() + cscale.bytes() + nzrows.bytes() + emptyrows.bytes() + rowptr_t.bytes() +
               colx.bytes() + colx_stage[0].bytes() + colx_stage[1].bytes() + segments.bytes() + fixups.bytes() + hubs.bytes() +
               scratch.bytes() + dev_error.bytes();
    for (const auto& s : slab) t += s.bytes();
    for (const auto& s : whole) t += s.bytes();
    return (int64_t)t;
}

int64_t gnnpre_plan::host_bytes() const { return (int64_t)colx_host.bytes(); }

namespace {

int build_plan_impl(const gnnpre_csr_t* csr, const int32_t* degrees, const gnnpre_plan_opts_t* opts,
                    gnnpre_plan* P) {
    const int64_t n = csr->n, nnz = csr->nnz;
    const bool diag = opts->op != GNNPRE_OP_SAGE_MEAN;
    cudaStream_t st = nullptr;  // the plan is built on the legacy default stream and synchronised
    GNNPRE_CUDA(cudaGetDevice(&P->device));
    P->n = n;
    P->nnz = nnz;
    P->nnz_tilde = nnz + (diag ? n : 0);
    P->feat_dim = (opts->feat_dim + 3) / 4 * 4;  // whole float4 columns; the caller's leading dimensions cover the pad
    P->op = opts->op;
    P->gin_eps = opts->gin_eps;
    P->teleport_alpha = opts->teleport_alpha;
    P->flags = opts->flags;
    P->structure_mem = csr->mem;
    const int64_t m = P->nnz_tilde;

    // ---- the CSR on the device (a temporary copy when the caller's lives on the host)
    DevBuf<int64_t> tmp_rowptr;
    DevBuf<int32_t> tmp_colidx, tmp_deg;
    const int64_t* d_rowptr = csr->rowptr;
    const int32_t* d_colidx = csr->colidx;
    const int32_t* d_deg_in = degrees;
    if (csr->mem == GNNPRE_MEM_HOST) {
        if (csr->rowptr[0] != 0 || csr->rowptr[n] != nnz) return GNNPRE_ERR_INVALID_CSR;
        GNNPRE_TRY(tmp_rowptr.alloc((size_t)n + 1));
        GNNPRE_TRY(tmp_colidx.alloc((size_t)nnz));
        GNNPRE_CUDA(cudaMemcpy(tmp_rowptr.p, csr->rowptr, sizeof(int64_t) * (size_t)(n + 1), cudaMemcpyHostToDevice));
        if (nnz) GNNPRE_CUDA(cudaMemcpy(tmp_colidx.p, csr->colidx, sizeof(int32_t) * (size_t)nnz, cudaMemcpyHostToDevice));
        d_rowptr = tmp_rowptr.p;
        d_colidx = tmp_colidx.p;
        if (degrees) {
            GNNPRE_TRY(tmp_deg.alloc((size_t)n));
            GNNPRE_CUDA(cudaMemcpy(tmp_deg.p, degrees, sizeof(int32_t) * (size_t)n, cudaMemcpyHostToDevice));
            d_deg_in = tmp_deg.p;
        }
    } else {
        int64_t ends[2] = {-1, -1};
        GNNPRE_CUDA(cudaMemcpy(&ends[0], csr->rowptr, sizeof(int64_t), cudaMemcpyDeviceToHost));
        GNNPRE_CUDA(cudaMemcpy(&ends[1], csr->rowptr + n, sizeof(int64_t), cudaMemcpyDeviceToHost));
        if (ends[0] != 0 || ends[1] != nnz) return GNNPRE_ERR_INVALID_CSR;
    }

    // ---- validation
    if (!(opts->flags & GNNPRE_FLAG_SKIP_VALIDATION)) {
        DevBuf<int> err;
        GNNPRE_TRY(err.alloc(1));
        GNNPRE_CUDA(cudaMemsetAsync(err.p, 0, sizeof(int), st));
        k_validate<<<grid_for(n * 32, kTB), kTB, 0, st>>>(n, nnz, d_rowptr, d_colidx, err.p);
        GNNPRE_CUDA(cudaGetLastError());
        int h = 0;
        GNNPRE_CUDA(cudaMemcpy(&h, err.p, sizeof(int), cudaMemcpyDeviceToHost));
        if (h) return GNNPRE_ERR_INVALID_CSR;
    }

    // ---- degrees and scales
    GNNPRE_TRY(P->deg.alloc((size_t)n));
    if (d_deg_in) {
        GNNPRE_CUDA(cudaMemcpyAsync(P->deg.p, d_deg_in, sizeof(int32_t) * (size_t)n, cudaMemcpyDeviceToDevice, st));
    } else {
        k_degrees<<<grid_for(n, kTB), kTB, 0, st>>>(n, d_rowptr, P->deg.p);
        GNNPRE_CUDA(cudaGetLastError());
    }
    GNNPRE_TRY(P->rscale.alloc((size_t)n));
    GNNPRE_TRY(P->cscale.alloc((size_t)n));
    k_scales<<<grid_for(n, kTB), kTB, 0, st>>>(P->op, n, P->deg.p, P->rscale.p, P->cscale.p);
    GNNPRE_CUDA(cudaGetLastError());

    // ---- E, the support's edge list
    GNNPRE_TRY(P->rowptr_t.alloc((size_t)n + 1));
    GNNPRE_TRY(P->colx.alloc((size_t)m));
    k_support<<<grid_for(n * 32, kTB), kTB, 0, st>>>(diag ? 1 : 0, n, d_rowptr, d_colidx, P->rowptr_t.p, P->colx.p);
    GNNPRE_CUDA(cudaGetLastError());
    GNNPRE_CUDA(cudaStreamSynchronize(st));
    tmp_colidx.reset();
    tmp_rowptr.reset();
    tmp_deg.reset();

    // ---- rows with / without edges (only SAGE can have empty rows)
    DevBuf<int32_t> rank;
    P->rows_all_nonempty = true;
    P->num_nonempty = n;
    P->num_empty = 0;
    if (!diag) {
        DevBuf<int32_t> flag;
        GNNPRE_TRY(flag.alloc((size_t)n));
        GNNPRE_TRY(rank.alloc((size_t)n + 1));
        k_nonempty_flags<<<grid_for(n, kTB), kTB, 0, st>>>(n, P->rowptr_t.p, flag.p);
        GNNPRE_CUDA(cudaGetLastError());
        GNNPRE_TRY(exclusive_scan(flag.p, n, rank.p, st));
        int32_t nonempty = 0;
        GNNPRE_CUDA(cudaMemcpy(&nonempty, rank.p + n, sizeof(int32_t), cudaMemcpyDeviceToHost));
        P->num_nonempty = nonempty;
        P->num_empty = n - nonempty;
        if (P->num_empty > 0) {
            P->rows_all_nonempty = false;
            GNNPRE_TRY(P->nzrows.alloc((size_t)P->num_nonempty));
            GNNPRE_TRY(P->emptyrows.alloc((size_t)P->num_empty));
            k_split_rows<<<grid_for(n, kTB), kTB, 0, st>>>(n, flag.p, rank.p, P->nzrows.p, P->emptyrows.p);
            GNNPRE_CUDA(cudaGetLastError());
            GNNPRE_CUDA(cudaStreamSynchronize(st));
        } else {
            rank.reset();
        }
    }

    // ---- Eq. 12: (b, c)
    const int64_t F = P->feat_dim;
    P->B_S = 4 * m + 8 * (n + 1);
    P->B_X = 4 * n * F;
    P->B_fixed = 16 * n;
    P->beta_S = csr->mem == GNNPRE_MEM_HOST ? 2 : 1;
    P->beta_X = opts->operands_mem == GNNPRE_MEM_HOST ? 4 : 2;
    P->budget_bytes = opts->budget_bytes;
    if (P->budget_bytes <= 0) {
        size_t free_b = 0, total_b = 0;
        GNNPRE_CUDA(cudaMemGetInfo(&free_b, &total_b));
        // what this plan already holds counts as part of the budget it is about to be charged for
        P->budget_bytes = (int64_t)free_b + P->device_bytes();
    }
    const int64_t max_c = (F + 3) / 4;
    const int64_t max_b = std::min<int64_t>(std::max<int64_t>(m, 1), 1 << 20);
    int64_t b = opts->force_blocks, c = opts->force_col_slabs;
    if (b < 0 || c < 0 || c > max_c) return GNNPRE_ERR_INVALID_ARG;
    P->col_slabs_forced = c > 0;
    if (b > 0 && b > m) return GNNPRE_ERR_INVALID_ARG;
    if (b == 0 || c == 0) {
        // a forced value pins that variable; the other is searched
        int64_t sb = 0, sc = 0;
        const int64_t lo_c = c ? c : 1, hi_c = c ? c : max_c;
        bool found = false;
        for (int64_t cc = lo_c; cc <= hi_c; ++cc) {
            int64_t tb = 0, tc = 0;
            // restrict the search to this c by scaling: solve with max_c = 1 on B_X / cc
            const int64_t x_part = (P->beta_X * P->B_X + cc - 1) / cc;
            int rc = solve_budget(P->B_S, 0, P->B_fixed + x_part, P->beta_S, 1, P->budget_bytes, max_b, 1, &tb, &tc);
            if (rc != GNNPRE_OK) continue;
            if (b > 0) {
                if (tb > b) continue;  // the forced b is too small for this c
                tb = b;
            }
            if (!found || tb * cc < sb * sc) {
                found = true;
                sb = tb;
                sc = cc;
            }
        }
        if (!found) return GNNPRE_ERR_BUDGET_TOO_SMALL;
        b = sb;
        c = sc;
        // Host-resident operands: Eq. 12's model charges every block product the same, but with copies
        // overlapped a second slab lets the upload of X and the first hop's kernels run side by side.
        // Two slabs are used when the budget alone asks for one and the row pieces stay >= 256 bytes
        // (narrower strided pieces travel the host link below full speed); below 256 columns only for
        // two equal slabs, so that the pieces also start on 128-byte lines.
        if (opts->force_col_slabs == 0 && opts->operands_mem == GNNPRE_MEM_HOST && c == 1 && F >= 128 &&
            (F % 8 == 0 || F >= 256))
            c = 2;
        // Likewise a single edge block would hold every output row back until the whole hop is done;
        // eight blocks let finished rows leave for the host while the rest of the hop computes.
        if (opts->force_blocks == 0 && b == 1) {
            // E fits the budget whole: it stays on the device even when the caller's CSR lives on the host
            P->structure_mem = GNNPRE_MEM_DEVICE;
            if (opts->operands_mem == GNNPRE_MEM_HOST && m >= (1 << 20)) b = 8;
        }
    }
    if (m == 0) b = 1;
    P->b = (int32_t)b;
    P->c = (int32_t)c;
    P->slab_width = 4 * ((F + 4 * c - 1) / (4 * c));
    if (P->slab_width * (c - 1) >= F) return GNNPRE_ERR_INVALID_ARG;  // a slab would be empty
    GNNPRE_CUDA(cudaDeviceGetAttribute(&P->num_sms, cudaDevAttrMultiProcessorCount, P->device));
    // edges one launch covers: a hop when everything is resident, one block when blocks are launched singly
    const bool per_block = (opts->flags & GNNPRE_FLAG_LAUNCH_PER_BLOCK) || opts->operands_mem == GNNPRE_MEM_HOST ||
                           P->structure_mem == GNNPRE_MEM_HOST;
    const int64_t m_launch = per_block ? m / b : m;
    P->segment_edges = opts->segment_edges > 0
                           ? opts->segment_edges
                           : auto_segment_edges(P->slab_width, m_launch, uses_bulk_copy(P, (int32_t)P->slab_width),
                                                P->num_sms);
    if (P->segment_edges < 1) return GNNPRE_ERR_INVALID_ARG;

    // ---- block table: block l = edges [floor(l m / b), floor((l+1) m / b))
    P->blocks.assign((size_t)b, Block{});
    std::vector<int64_t> e_off((size_t)b + 1), seg_base((size_t)b + 1);
    {
        const int64_t q = m / b, r = m % b;
        for (int64_t l = 0; l <= b; ++l) e_off[(size_t)l] = l * q + (l * r) / b;
    }
    const int32_t L = P->segment_edges;
    seg_base[0] = 0;
    for (int64_t l = 0; l < b; ++l)
        seg_base[(size_t)l + 1] = seg_base[(size_t)l] + (e_off[(size_t)l + 1] - e_off[(size_t)l] + L - 1) / L;
    const int64_t nseg = seg_base[(size_t)b];
    if (nseg >= 0x3fffffffLL) return GNNPRE_ERR_INVALID_ARG;
    P->num_segments = nseg;
    GNNPRE_TRY(P->segments.alloc((size_t)nseg + 1));
    if (m == 0) {
        // no edges at all: every row is empty; one empty block
        P->blocks[0] = Block{0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, n};
        Segment sentinel{0, 0, -1, -1, 0};
        GNNPRE_CUDA(cudaMemcpy(P->segments.p, &sentinel, sizeof(Segment), cudaMemcpyHostToDevice));
        return GNNPRE_OK;
    }

    DevBuf<int64_t> d_e_off, d_seg_base;
    GNNPRE_TRY(d_e_off.alloc((size_t)b + 1));
    GNNPRE_TRY(d_seg_base.alloc((size_t)b + 1));
    GNNPRE_CUDA(cudaMemcpy(d_e_off.p, e_off.data(), sizeof(int64_t) * (size_t)(b + 1), cudaMemcpyHostToDevice));
    GNNPRE_CUDA(cudaMemcpy(d_seg_base.p, seg_base.data(), sizeof(int64_t) * (size_t)(b + 1), cudaMemcpyHostToDevice));

    DevBuf<BlockRows> d_rows;
    GNNPRE_TRY(d_rows.alloc((size_t)b));
    k_block_rows<<<grid_for(b, kTB), kTB, 0, st>>>((int)b, d_e_off.p, P->rowptr_t.p, n, d_rows.p);
    GNNPRE_CUDA(cudaGetLastError());
    std::vector<BlockRows> h_rows((size_t)b);
    GNNPRE_CUDA(cudaMemcpy(h_rows.data(), d_rows.p, sizeof(BlockRows) * (size_t)b, cudaMemcpyDeviceToHost));

    // ---- segments, scratch slots and row fix-ups
    // How far a nominal cut inside a row may move forward to the next row start.  Half a segment keeps the segments
    // balanced (moving by up to a whole one cost 3-15 % on every larger workload).  A launch so small that all its
    // segments are resident at once is bound by latency, not balance: there the cut may move by up to L - 1 edges,
    // which leaves a graph of short rows without any cut row and so without the fix-up launch (4,096 nodes of
    // degree 16: two launches per step of two hops instead of four, 39 -> 31 us).
    const int64_t f4_slab = std::min<int64_t>(P->slab_width, 512) / 4;
    const int64_t lanes = f4_slab <= 4 ? 4 : f4_slab <= 8 ? 8 : f4_slab <= 16 ? 16 : 32;
    const bool one_wave = nseg * lanes <= (int64_t)P->num_sms * 768;
    const int32_t snap = one_wave ? L - 1 : L / 2;
    k_segment_starts<<<grid_for(nseg + 1, kTB), kTB, 0, st>>>(nseg, (int)b, d_seg_base.p, d_e_off.p, L, snap,
                                                              P->rowptr_t.p, n, rank.p, P->segments.p);
    GNNPRE_CUDA(cudaGetLastError());
    DevBuf<int32_t> flags, slot_scan, emit, emit_scan;
    GNNPRE_TRY(flags.alloc((size_t)nseg * 2));
    GNNPRE_TRY(slot_scan.alloc((size_t)nseg * 2 + 1));
    GNNPRE_TRY(emit.alloc((size_t)nseg));
    GNNPRE_TRY(emit_scan.alloc((size_t)nseg + 1));
    k_segment_flags<<<grid_for(nseg, kTB), kTB, 0, st>>>(nseg, P->segments.p, P->rowptr_t.p, flags.p, emit.p);
    GNNPRE_CUDA(cudaGetLastError());
    GNNPRE_TRY(exclusive_scan(flags.p, nseg * 2, slot_scan.p, st));
    GNNPRE_TRY(exclusive_scan(emit.p, nseg, emit_scan.p, st));
    int32_t n_slots = 0, n_fix = 0;
    GNNPRE_CUDA(cudaMemcpy(&n_slots, slot_scan.p + nseg * 2, sizeof(int32_t), cudaMemcpyDeviceToHost));
    GNNPRE_CUDA(cudaMemcpy(&n_fix, emit_scan.p + nseg, sizeof(int32_t), cudaMemcpyDeviceToHost));
    P->num_slots = n_slots;
    P->num_fixups = n_fix;
    GNNPRE_TRY(P->fixups.alloc((size_t)n_fix));
    k_segment_finalize<<<grid_for(nseg, kTB), kTB, 0, st>>>(nseg, P->segments.p, P->rowptr_t.p, flags.p, slot_scan.p,
                                                            emit.p, emit_scan.p, P->fixups.p);
    GNNPRE_CUDA(cudaGetLastError());
    k_clear_pad<<<grid_for(nseg + 1, kTB), kTB, 0, st>>>(nseg, P->segments.p);
    GNNPRE_CUDA(cudaGetLastError());

    // fix-up ranges per block: the scan value at each block's first segment
    DevBuf<int32_t> d_fix_at;
    GNNPRE_TRY(d_fix_at.alloc((size_t)b + 1));
    k_gather_i32<<<grid_for(b + 1, kTB), kTB, 0, st>>>((int)(b + 1), d_seg_base.p, emit_scan.p, d_fix_at.p);
    GNNPRE_CUDA(cudaGetLastError());
    std::vector<int32_t> fix_at((size_t)b + 1);
    GNNPRE_CUDA(cudaMemcpy(fix_at.data(), d_fix_at.p, sizeof(int32_t) * (size_t)(b + 1), cudaMemcpyDeviceToHost));

    // hub rows (more parts than a warp adds quickly) are listed so that the fix-up kernel can give each a CTA
    P->hub_parts = hub_parts_for(P->slab_width);
    std::vector<int32_t> hub_at((size_t)b + 1, 0);
    if (n_fix > 0) {
        DevBuf<int32_t> hub_flag, hub_scan, d_hub_at;
        DevBuf<int64_t> d_fix_at64;
        GNNPRE_TRY(hub_flag.alloc((size_t)n_fix));
        GNNPRE_TRY(hub_scan.alloc((size_t)n_fix + 1));
        k_hub_flags<<<grid_for(n_fix, kTB), kTB, 0, st>>>(n_fix, P->fixups.p, P->hub_parts, hub_flag.p);
        GNNPRE_CUDA(cudaGetLastError());
        GNNPRE_TRY(exclusive_scan(hub_flag.p, n_fix, hub_scan.p, st));
        int32_t n_hubs = 0;
        GNNPRE_CUDA(cudaMemcpy(&n_hubs, hub_scan.p + n_fix, sizeof(int32_t), cudaMemcpyDeviceToHost));
        P->num_hubs = n_hubs;
        if (n_hubs > 0) {
            GNNPRE_TRY(P->hubs.alloc((size_t)n_hubs));
            k_hub_scatter<<<grid_for(n_fix, kTB), kTB, 0, st>>>(n_fix, hub_flag.p, hub_scan.p, P->hubs.p);
            GNNPRE_CUDA(cudaGetLastError());
            std::vector<int64_t> fix_at64(fix_at.begin(), fix_at.end());
            GNNPRE_TRY(d_fix_at64.alloc((size_t)b + 1));
            GNNPRE_TRY(d_hub_at.alloc((size_t)b + 1));
            GNNPRE_CUDA(cudaMemcpy(d_fix_at64.p, fix_at64.data(), sizeof(int64_t) * (size_t)(b + 1), cudaMemcpyHostToDevice));
            k_gather_i32<<<grid_for(b + 1, kTB), kTB, 0, st>>>((int)(b + 1), d_fix_at64.p, hub_scan.p, d_hub_at.p);
            GNNPRE_CUDA(cudaGetLastError());
            GNNPRE_CUDA(cudaMemcpy(hub_at.data(), d_hub_at.p, sizeof(int32_t) * (size_t)(b + 1), cudaMemcpyDeviceToHost));
        }
        GNNPRE_CUDA(cudaStreamSynchronize(st));  // temporaries die here
    }

    for (int64_t l = 0; l < b; ++l) {
        Block& B = P->blocks[(size_t)l];
        const BlockRows& r = h_rows[(size_t)l];
        B.e_lo = e_off[(size_t)l];
        B.e_hi = e_off[(size_t)l + 1];
        B.row_lo = r.row_lo;
        B.row_hi = r.row_hi;
        B.first_partial = r.first_partial;
        B.last_partial = r.last_partial;
        B.seg_lo = seg_base[(size_t)l];
        B.seg_hi = seg_base[(size_t)l + 1];
        B.fix_lo = fix_at[(size_t)l];
        B.fix_hi = fix_at[(size_t)l + 1];
        B.hub_lo = hub_at[(size_t)l];
        B.hub_hi = hub_at[(size_t)l + 1];
        B.done_row_lo = l == 0 ? 0 : h_rows[(size_t)l - 1].done_row_hi;
        B.done_row_hi = l == b - 1 ? n : r.done_row_hi;
    }

    GNNPRE_TRY(P->scratch.alloc((size_t)P->num_slots * (size_t)P->slab_width));
    GNNPRE_TRY(P->dev_error.alloc(1));
    GNNPRE_CUDA(cudaMemset(P->dev_error.p, 0, sizeof(int)));

    // ---- a host-resident structure keeps E in pinned memory and streams it block by block
    if (P->structure_mem == GNNPRE_MEM_HOST) {
        GNNPRE_TRY(P->colx_host.alloc((size_t)m));
        GNNPRE_CUDA(cudaMemcpy(P->colx_host.p, P->colx.p, sizeof(uint32_t) * (size_t)m, cudaMemcpyDeviceToHost));
        P->colx.reset();
        int64_t longest = 0;
        for (const Block& B : P->blocks) longest = std::max(longest, B.e_hi - B.e_lo);
        GNNPRE_TRY(P->colx_stage[0].alloc((size_t)longest));
        if (b > 1) GNNPRE_TRY(P->colx_stage[1].alloc((size_t)longest));
    }
    GNNPRE_CUDA(cudaStreamSynchronize(st));
    return GNNPRE_OK;
}

}  // namespace

extern "C" int gnnpre_degrees(const gnnpre_csr_t* csr, int32_t* deg_out, void* stream) {
    if (!csr || !deg_out || !csr->rowptr || csr->n < 0) return GNNPRE_ERR_INVALID_ARG;
    GNNPRE_TRY(check_device());
    const int64_t n = csr->n;
    if (n == 0) return GNNPRE_OK;
    cudaStream_t st = (cudaStream_t)stream;
    if (csr->mem == GNNPRE_MEM_DEVICE) {
        k_degrees<<<grid_for(n, kTB), kTB, 0, st>>>(n, csr->rowptr, deg_out);
        GNNPRE_CUDA(cudaGetLastError());
        return GNNPRE_OK;
    }
    DevBuf<int64_t> rp;
    DevBuf<int32_t> dg;
    GNNPRE_TRY(rp.alloc((size_t)n + 1));
    GNNPRE_TRY(dg.alloc((size_t)n));
    GNNPRE_CUDA(cudaMemcpyAsync(rp.p, csr->rowptr, sizeof(int64_t) * (size_t)(n + 1), cudaMemcpyHostToDevice, st));
    k_degrees<<<grid_for(n, kTB), kTB, 0, st>>>(n, rp.p, dg.p);
    GNNPRE_CUDA(cudaGetLastError());
    GNNPRE_CUDA(cudaMemcpyAsync(deg_out, dg.p, sizeof(int32_t) * (size_t)n, cudaMemcpyDeviceToHost, st));
    GNNPRE_CUDA(cudaStreamSynchronize(st));
    return GNNPRE_OK;
}

extern "C" int gnnpre_build_plan(const gnnpre_csr_t* csr, const int32_t* degrees, const gnnpre_plan_opts_t* opts,
                                 gnnpre_plan_t** plan_out) {
    if (!csr || !opts || !plan_out) return GNNPRE_ERR_INVALID_ARG;
    *plan_out = nullptr;
    if (csr->n < 1 || csr->n >= 0x7fffffffLL || csr->nnz < 0 || !csr->rowptr || (csr->nnz > 0 && !csr->colidx))
        return GNNPRE_ERR_INVALID_ARG;
    if (csr->mem != GNNPRE_MEM_DEVICE && csr->mem != GNNPRE_MEM_HOST) return GNNPRE_ERR_INVALID_ARG;
    if (opts->op < GNNPRE_OP_GCN_SYM || opts->op > GNNPRE_OP_GIN_SUM) return GNNPRE_ERR_INVALID_ARG;
    if (opts->operands_mem != GNNPRE_MEM_DEVICE && opts->operands_mem != GNNPRE_MEM_HOST) return GNNPRE_ERR_INVALID_ARG;
    if (!(opts->teleport_alpha >= 0.f && opts->teleport_alpha <= 1.f)) return GNNPRE_ERR_INVALID_ARG;
    if (opts->feat_dim < 1) return GNNPRE_ERR_INVALID_ARG;
    if (opts->segment_edges < 0 || opts->segment_edges > (1 << 20)) return GNNPRE_ERR_INVALID_ARG;
    GNNPRE_TRY(check_device());
    gnnpre_plan* P = new (std::nothrow) gnnpre_plan();
    if (!P) return GNNPRE_ERR_OOM_HOST;
    int rc = build_plan_impl(csr, degrees, opts, P);
    if (rc != GNNPRE_OK) {
        delete P;
        return rc;
    }
    *plan_out = P;
    return GNNPRE_OK;
}

extern "C" int gnnpre_plan_info(const gnnpre_plan_t* P, gnnpre_plan_info_t* o) {
    if (!P || !o) return GNNPRE_ERR_INVALID_ARG;
    std::memset(o, 0, sizeof(*o));
    o->n = P->n;
    o->nnz = P->nnz;
    o->nnz_tilde = P->nnz_tilde;
    o->feat_dim = P->feat_dim;
    o->op = P->op;
    o->b = P->b;
    o->c = P->c;
    o->slab_width = P->slab_width;
    o->B_S = P->B_S;
    o->B_X = P->B_X;
    o->B_fixed = P->B_fixed;
    o->beta_S = P->beta_S;
    o->beta_X = P->beta_X;
    o->budget_bytes = P->budget_bytes;
    o->device_bytes = P->device_bytes();
    o->host_bytes = P->host_bytes();
    o->num_segments = P->num_segments;
    o->num_row_fixups = P->num_fixups;
    o->num_scratch_rows = P->num_slots;
    o->segment_edges = P->segment_edges;
    o->structure_mem = P->structure_mem;
    return GNNPRE_OK;
}

extern "C" int gnnpre_plan_block(const gnnpre_plan_t* P, int32_t l, gnnpre_block_info_t* o) {
    if (!P || !o || l < 0 || l >= P->b) return GNNPRE_ERR_INVALID_ARG;
    const Block& B = P->blocks[(size_t)l];
    o->e_lo = B.e_lo;
    o->e_hi = B.e_hi;
    o->row_lo = B.row_lo;
    o->row_hi = B.row_hi;
    o->first_row_partial = B.first_partial;
    o->last_row_partial = B.last_partial;
    return GNNPRE_OK;
}

extern "C" int gnnpre_plan_scales(const gnnpre_plan_t* P, int32_t* deg_out, float* rscale_out, float* cscale_out) {
    if (!P) return GNNPRE_ERR_INVALID_ARG;
    const size_t n = (size_t)P->n;
    if (deg_out) GNNPRE_CUDA(cudaMemcpy(deg_out, P->deg.p, sizeof(int32_t) * n, cudaMemcpyDeviceToHost));
    if (rscale_out) GNNPRE_CUDA(cudaMemcpy(rscale_out, P->rscale.p, sizeof(float) * n, cudaMemcpyDeviceToHost));
    if (cscale_out) GNNPRE_CUDA(cudaMemcpy(cscale_out, P->cscale.p, sizeof(float) * n, cudaMemcpyDeviceToHost));
    return GNNPRE_OK;
}

extern "C" int gnnpre_plan_support(const gnnpre_plan_t* P, int64_t* rowptr_out, int32_t* colidx_out) {
    if (!P) return GNNPRE_ERR_INVALID_ARG;
    if (rowptr_out)
        GNNPRE_CUDA(cudaMemcpy(rowptr_out, P->rowptr_t.p, sizeof(int64_t) * (size_t)(P->n + 1), cudaMemcpyDeviceToHost));
    if (colidx_out && P->nnz_tilde > 0) {
        const size_t m = (size_t)P->nnz_tilde;
        if (P->structure_mem == GNNPRE_MEM_HOST) {
            std::memcpy(colidx_out, P->colx_host.p, sizeof(uint32_t) * m);
        } else {
            GNNPRE_CUDA(cudaMemcpy(colidx_out, P->colx.p, sizeof(uint32_t) * m, cudaMemcpyDeviceToHost));
        }
        for (size_t e = 0; e < m; ++e) colidx_out[e] &= 0x7fffffff;  // drop the row-end marks
    }
    return GNNPRE_OK;
}

extern "C" void gnnpre_plan_destroy(gnnpre_plan_t* P) {
    if (!P) return;
    // Wait for the work that still uses the plan's memory - the last device-resident call (an event on the
    // caller's stream) and the plan's own streams - not for the whole device.
    // (an event last recorded inside a stream capture cannot be waited for: then wait for the device)
    if (P->last_use && cudaEventSynchronize(P->last_use) != cudaSuccess) {
        (void)cudaGetLastError();
        cudaDeviceSynchronize();
    }
    if (P->s_h2d) cudaStreamSynchronize(P->s_h2d);
    if (P->s_compute) cudaStreamSynchronize(P->s_compute);
    if (P->s_d2h) cudaStreamSynchronize(P->s_d2h);
    if (P->s_struct) cudaStreamSynchronize(P->s_struct);
    (void)cudaGetLastError();
    delete P;
}

extern "C" int gnnpre_solve_budget(int64_t B_S, int64_t B_X, int64_t B_fixed, int64_t beta_S, int64_t beta_X,
                                   int64_t B_GPU, int64_t max_b, int64_t max_c, int64_t* b_out, int64_t* c_out) {
    if (!b_out || !c_out) return GNNPRE_ERR_INVALID_ARG;
    return solve_budget(B_S, B_X, B_fixed, beta_S, beta_X, B_GPU, max_b, max_c, b_out, c_out);
}
