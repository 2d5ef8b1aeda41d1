// Propagation kernels: one hop  X_out = A^ X_prev  over a range of warp-level edge segments
// (Algorithm 1's block product Z = S^(j) X^(i) and its accumulation X_tmp += Z, fused; the
// operator's normalisation of Eq. 1 / Eq. 10 is applied on the fly from per-node scales, so S is
// never materialised).
//
// Work decomposition.  The edge list E of the support is cut, inside every edge block, into short
// contiguous segments.  A group of G lanes (G = 4..32, so that one lane holds one or more float4 of
// a feature row) walks one segment edge by edge: the group reads up to G column indices with one
// coalesced load, then gathers the neighbours' feature rows with 128-bit loads, several rows in
// flight per lane, and accumulates in fp32 registers.  Bit 31 of a column entry marks the last edge
// of a row: there the group scales the sum by r_i and stores the output row.  Rows cut by a segment
// boundary leave their partial sums in scratch rows, which k_row_fixups adds up in a fixed order.
#include <algorithm>
#include <atomic>

#include "gnnpre_internal.cuh"

namespace gnnpre {

namespace {

#include "segments_common.cuh"
#include "segments.cuh"
#include "segments_tma.cuh"

// A wait on a barrier that nothing ever completes: the polls run out, the error word is set, the warp
// leaves.  This is the give-up path of k_segments_tma, exercised on its own.
__global__ void k_wait_that_runs_out(int* error, uint32_t polls) {
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    bool done = false;
    for (uint32_t i = 0; i < polls && !done; ++i) done = mbar_try_wait(b, 0);
    if (!done && threadIdx.x == 0) atomicExch(error, 1);
}

#include "fixups.cuh"
#include "ceiling.cuh"

template <int G, int V, int U>
int launch_segments_shape(const gnnpre_plan* P, const SegArgs& a, cudaStream_t st) {
    const int64_t groups = a.seg_hi - a.seg_lo;
    const unsigned grid = (unsigned)((groups * G + kThreads - 1) / kThreads);
    const int ep = epilogue_of(a.tp);
#define GNNPRE_LAUNCH_SEGMENTS(OP_, EMPTY_)                                                                 \
    do {                                                                                                    \
        if (ep == kEpSum) k_segments<G, V, U, OP_, EMPTY_, kEpSum><<<grid, kThreads, 0, st>>>(a);           \
        else if (ep == kEpTeleport) k_segments<G, V, U, OP_, EMPTY_, kEpTeleport><<<grid, kThreads, 0, st>>>(a); \
        else k_segments<G, V, U, OP_, EMPTY_, kEpPlain><<<grid, kThreads, 0, st>>>(a);                      \
    } while (0)
    switch (P->op) {
    case GNNPRE_OP_GCN_SYM: GNNPRE_LAUNCH_SEGMENTS(GNNPRE_OP_GCN_SYM, false); break;
    case GNNPRE_OP_GIN_SUM: GNNPRE_LAUNCH_SEGMENTS(GNNPRE_OP_GIN_SUM, false); break;
    default:
        if (P->rows_all_nonempty) GNNPRE_LAUNCH_SEGMENTS(GNNPRE_OP_SAGE_MEAN, false);
        else GNNPRE_LAUNCH_SEGMENTS(GNNPRE_OP_SAGE_MEAN, true);
    }
#undef GNNPRE_LAUNCH_SEGMENTS
    GNNPRE_CUDA(cudaGetLastError());
    return GNNPRE_OK;
}

// Bulk-copy variant: one persistent CTA per SM, as many warps (at most kTmaMaxWarps) as fit into the
// SM's shared memory with kTmaStages stages of kTmaRows rows each.
constexpr size_t kTmaSmemBudget = 227 * 1024 - 1024;

uint32_t tma_stage_bytes(int32_t f4) { return (kTmaRows / 4) * ((4u * 16u * (uint32_t)f4 + 127u) & ~127u); }

int tma_warps(int32_t f4) {
    const size_t per_warp = (size_t)kTmaStages * tma_stage_bytes(f4);
    return (int)std::min<size_t>(kTmaMaxWarps, kTmaSmemBudget / per_warp);
}

// Tensor map of the [n, width] fp32 matrix at `x` with row stride ldx: box = one row of `width` columns,
// no swizzle, no interleave.  The driver entry point is looked up once (no link-time dependency on libcuda).
int make_row_tensor_map(const float* x, int64_t n, int32_t width, int64_t ldx, CUtensorMap* out) {
    typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static std::atomic<encode_fn> cached{nullptr};  // threads may race to fill it; they all store the same pointer
    encode_fn encode = cached.load(std::memory_order_acquire);
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        GNNPRE_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (q != cudaDriverEntryPointSuccess || !fn) return GNNPRE_ERR_CUDA;
        encode = reinterpret_cast<encode_fn>(fn);
        cached.store(encode, std::memory_order_release);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)width, (cuuint64_t)n};
    const cuuint64_t strides[1] = {(cuuint64_t)ldx * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)width, 1u};
    const cuuint32_t elem[2] = {1u, 1u};
    const CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(x), dims, strides, box, elem,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled", __FILE__, __LINE__);
        return GNNPRE_ERR_CUDA;
    }
    return GNNPRE_OK;
}

// The plan remembers the tensor maps of the matrices it has met (a K-hop call alternates between a few), so a
// launch in steady state encodes nothing.
int cached_tensor_map(const gnnpre_plan* P, const SegArgs& a, const CUtensorMap** out) {
    for (const auto& c : P->tmaps) {
        if (c.x == a.x && c.ldx == a.ldx && c.f4 == a.f4) {
            *out = &c.map;
            return GNNPRE_OK;
        }
    }
    if (P->tmaps.size() >= 32) P->tmaps.erase(P->tmaps.begin());
    gnnpre_plan::TensorMapEntry entry;
    entry.x = a.x;
    entry.ldx = a.ldx;
    entry.f4 = a.f4;
    GNNPRE_TRY(make_row_tensor_map(a.x, P->n, 4 * a.f4, a.ldx, &entry.map));
    P->tmaps.push_back(entry);
    *out = &P->tmaps.back().map;
    return GNNPRE_OK;
}

template <int OP, bool HAS_EMPTY, int F4C, int EP>
int launch_segments_tma_width(const gnnpre_plan* P, const SegArgs& a, cudaStream_t st) {
    const int nwarps = tma_warps(a.f4);
    const size_t smem = (size_t)nwarps * kTmaStages * tma_stage_bytes(a.f4);
    const CUtensorMap* tmap = nullptr;
    GNNPRE_TRY(cached_tensor_map(P, a, &tmap));
    auto kernel = k_segments_tma<OP, HAS_EMPTY, F4C, EP>;
    // the opt-in to large dynamic shared memory is per kernel and device: once, and again only if a launch needs more
    static std::atomic<int> smem_set[kMaxDevices];
    const int dev = P->device < kMaxDevices ? P->device : 0;
    if (P->device >= kMaxDevices || smem_set[dev].load(std::memory_order_relaxed) < (int)smem) {
        GNNPRE_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        smem_set[dev].store((int)smem, std::memory_order_relaxed);
    }
    const int64_t nseg = a.seg_hi - a.seg_lo;
    const unsigned grid = (unsigned)std::min<int64_t>(P->num_sms, (nseg + nwarps - 1) / nwarps);
    kernel<<<grid, nwarps * 32, smem, st>>>(a, *tmap, P->dev_error.p);
    GNNPRE_CUDA(cudaGetLastError());
    return GNNPRE_OK;
}

// Rows (or column tiles) of 100 and of 128 columns get kernels with the row size compiled in.
template <int OP, bool HAS_EMPTY>
int launch_segments_tma_op(const gnnpre_plan* P, const SegArgs& a, cudaStream_t st) {
    const int ep = epilogue_of(a.tp);
    if (ep == kEpSum) return launch_segments_tma_width<OP, HAS_EMPTY, 0, kEpSum>(P, a, st);
    if (ep == kEpTeleport) return launch_segments_tma_width<OP, HAS_EMPTY, 0, kEpTeleport>(P, a, st);
    if (a.f4 == 25) return launch_segments_tma_width<OP, HAS_EMPTY, 25, kEpPlain>(P, a, st);
    if (a.f4 == 32) return launch_segments_tma_width<OP, HAS_EMPTY, 32, kEpPlain>(P, a, st);
    return launch_segments_tma_width<OP, HAS_EMPTY, 0, kEpPlain>(P, a, st);
}

int launch_segments_tma(const gnnpre_plan* P, const SegArgs& a, cudaStream_t st) {
    switch (P->op) {
    case GNNPRE_OP_GCN_SYM: return launch_segments_tma_op<GNNPRE_OP_GCN_SYM, false>(P, a, st);
    case GNNPRE_OP_GIN_SUM: return launch_segments_tma_op<GNNPRE_OP_GIN_SUM, false>(P, a, st);
    default:
        return P->rows_all_nonempty ? launch_segments_tma_op<GNNPRE_OP_SAGE_MEAN, false>(P, a, st)
                                    : launch_segments_tma_op<GNNPRE_OP_SAGE_MEAN, true>(P, a, st);
    }
}

template <int G, int V>
int launch_fixups_shape(const FixArgs& a, cudaStream_t st) {
    const int64_t rows_per_cta = kThreads / 32;
    const unsigned grid = (unsigned)((a.hub_hi - a.hub_lo) + (a.fix_hi - a.fix_lo + rows_per_cta - 1) / rows_per_cta);
    const int ep = epilogue_of(a.tp);
    if (ep == kEpSum) k_row_fixups<G, V, kEpSum><<<grid, kThreads, 0, st>>>(a);
    else if (ep == kEpTeleport) k_row_fixups<G, V, kEpTeleport><<<grid, kThreads, 0, st>>>(a);
    else k_row_fixups<G, V, kEpPlain><<<grid, kThreads, 0, st>>>(a);
    GNNPRE_CUDA(cudaGetLastError());
    return GNNPRE_OK;
}

constexpr int kMaxTile = 512;  // columns one launch covers (G = 32, V = 4)

Teleport teleport_of(const gnnpre_plan* P, const HopArgs& h, int32_t f0) {
    Teleport tp;
    tp.x0 = h.x0 ? h.x0 + f0 : nullptr;
    tp.ldx0 = h.ldx0;
    tp.alpha = h.x0 ? P->teleport_alpha : 0.f;
    tp.keep = (float)(1.0 - (double)tp.alpha);
    tp.zsum = h.zsum ? h.zsum + f0 : nullptr;
    tp.ldz = h.ldz;
    tp.gamma = h.gamma;
    tp.gamma0 = h.gamma0;
    tp.zsum_first = h.zsum_first ? 1 : 0;
    return tp;
}

}  // namespace

namespace {

// A column tile of 68..128 columns (17..32 float4) goes through the bulk-copy kernel unless the plan says otherwise.
bool tile_uses_bulk_copy(const gnnpre_plan* P, int32_t width) {
    const int32_t f4 = width / 4;
    return !(P->flags & GNNPRE_FLAG_NO_BULK_COPY) && f4 > 16 && f4 <= 32 && tma_warps(f4) >= 2;
}

// Columns one segment launch covers.  Rows wider than 256 columns are cut into 128-column tiles for the bulk-copy
// kernel: the register kernel holds only two such rows per lane in flight (F = 602 on 23 M edges: 8.4 TB/s of
// gathered bytes for its 512-column tile against 11 TB/s for the copy engine on the rest of the row).
// Rows of 132..256 columns go the same way, as two equal tiles, once a 128-column tile of X no longer fits the
// L2 (2.4 M nodes, 124 M edges, F = 256: 11.9 ms per hop-launch on the register kernel plus 1.6 ms of fix-ups for
// its 128-edge segments, against 2 x 4.7 ms); while it fits, the register kernel's four rows per lane are the
// faster path (169 K nodes, F = 256: 0.25 ms against 2 x 0.15 ms).
int64_t l2_cache_bytes() {
    static int64_t cached = -1;
    if (cached < 0) {
        int dev = 0, bytes = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&bytes, cudaDevAttrL2CacheSize, dev) != cudaSuccess || bytes <= 0)
            bytes = 126 << 20;
        cached = bytes;
    }
    return cached;
}

int32_t segment_tile_width(const gnnpre_plan* P, int32_t width) {
    if (!tile_uses_bulk_copy(P, 128)) return kMaxTile;
    if (width > 256) return 128;
    if (width > 128 && P->n * 512 > l2_cache_bytes()) return 4 * ((width / 4 + 1) / 2);
    return kMaxTile;
}

}  // namespace

// Whether a slab of this width is (mostly) summed by the bulk-copy kernel; the plan sizes its segments for it.
bool uses_bulk_copy(const gnnpre_plan* P, int32_t width) {
    return tile_uses_bulk_copy(P, std::min(width, segment_tile_width(P, width)));
}

int launch_segments(const gnnpre_plan* P, const HopArgs& h, int64_t seg_lo, int64_t seg_hi, cudaStream_t st) {
    if (seg_hi <= seg_lo) return GNNPRE_OK;
    const int32_t tile = segment_tile_width(P, h.width);
    for (int32_t f0 = 0; f0 < h.width; f0 += tile) {
        const int32_t w = std::min<int32_t>(tile, h.width - f0);
        SegArgs a;
        a.segs = P->segments.p;
        a.seg_lo = seg_lo;
        a.seg_hi = seg_hi;
        a.colx = h.colx;
        a.colx_base = h.colx_edge_base;
        a.x = h.xprev + f0;
        a.ldx = h.ldx;
        a.out = h.xout + f0;
        a.ldo = h.ldo;
        a.scratch = P->scratch.p + f0;
        a.scratch_ld = P->slab_width;
        a.rscale = P->rscale.p;
        a.cscale = P->cscale.p;
        a.nzrows = P->nzrows.p;
        a.f4 = w / 4;
        a.diag_weight = 1.0f + P->gin_eps;
        a.tp = teleport_of(P, h, f0);
        if (tile_uses_bulk_copy(P, w)) GNNPRE_TRY(launch_segments_tma(P, a, st));
        else if (a.f4 <= 4) GNNPRE_TRY((launch_segments_shape<4, 1, 4>(P, a, st)));
        else if (a.f4 <= 8) GNNPRE_TRY((launch_segments_shape<8, 1, 8>(P, a, st)));
        else if (a.f4 <= 16) GNNPRE_TRY((launch_segments_shape<16, 1, 8>(P, a, st)));
        else if (a.f4 <= 32) GNNPRE_TRY((launch_segments_shape<32, 1, GNNPRE_SEG_U>(P, a, st)));
        else if (a.f4 <= 64) GNNPRE_TRY((launch_segments_shape<32, 2, 4>(P, a, st)));
        else GNNPRE_TRY((launch_segments_shape<32, 4, 2>(P, a, st)));
    }
    return GNNPRE_OK;
}

int launch_fixups(const gnnpre_plan* P, const HopArgs& h, int64_t fix_lo, int64_t fix_hi, int64_t hub_lo, int64_t hub_hi,
                  cudaStream_t st) {
    if (fix_hi <= fix_lo) return GNNPRE_OK;
    for (int32_t f0 = 0; f0 < h.width; f0 += kMaxTile) {
        const int32_t w = std::min<int32_t>(kMaxTile, h.width - f0);
        FixArgs a;
        a.fix = P->fixups.p;
        a.fix_lo = fix_lo;
        a.fix_hi = fix_hi;
        a.hubs = P->hubs.p;
        a.hub_lo = hub_lo;
        a.hub_hi = hub_hi;
        a.hub_parts = P->hub_parts;
        a.scratch = P->scratch.p + f0;
        a.scratch_ld = P->slab_width;
        a.rscale = P->rscale.p;
        a.out = h.xout + f0;
        a.ldo = h.ldo;
        a.f4 = w / 4;
        a.tp = teleport_of(P, h, f0);
        if (a.f4 <= 4) GNNPRE_TRY((launch_fixups_shape<4, 1>(a, st)));
        else if (a.f4 <= 8) GNNPRE_TRY((launch_fixups_shape<8, 1>(a, st)));
        else if (a.f4 <= 16) GNNPRE_TRY((launch_fixups_shape<16, 1>(a, st)));
        else if (a.f4 <= 32) GNNPRE_TRY((launch_fixups_shape<32, 1>(a, st)));
        else if (a.f4 <= 64) GNNPRE_TRY((launch_fixups_shape<32, 2>(a, st)));
        else GNNPRE_TRY((launch_fixups_shape<32, 4>(a, st)));
    }
    return GNNPRE_OK;
}

int launch_zero_empty_rows(const gnnpre_plan* P, const HopArgs& h, cudaStream_t st) {
    if (P->num_empty == 0) return GNNPRE_OK;
    const int32_t f4 = h.width / 4;
    const int64_t items = P->num_empty * f4;
    const Teleport tp = teleport_of(P, h, 0);
    const unsigned grid = (unsigned)((items + 255) / 256);
    const int ep = epilogue_of(tp);
    if (ep == kEpSum) k_zero_rows<kEpSum><<<grid, 256, 0, st>>>(P->emptyrows.p, P->num_empty, h.xout, h.ldo, f4, tp);
    else if (ep == kEpTeleport) k_zero_rows<kEpTeleport><<<grid, 256, 0, st>>>(P->emptyrows.p, P->num_empty, h.xout, h.ldo, f4, tp);
    else k_zero_rows<kEpPlain><<<grid, 256, 0, st>>>(P->emptyrows.p, P->num_empty, h.xout, h.ldo, f4, tp);
    GNNPRE_CUDA(cudaGetLastError());
    return GNNPRE_OK;
}

namespace {

template <int F4C>
int launch_ceiling_tma(const gnnpre_plan* P, const SegArgs& a, float* sink, cudaStream_t st) {
    const int nwarps = tma_warps(a.f4);
    const size_t smem = (size_t)nwarps * kTmaStages * tma_stage_bytes(a.f4);
    const CUtensorMap* tmap = nullptr;
    GNNPRE_TRY(cached_tensor_map(P, a, &tmap));
    auto kernel = k_ceiling_tma<F4C>;
    GNNPRE_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int64_t nseg = a.seg_hi - a.seg_lo;
    const unsigned grid = (unsigned)std::min<int64_t>(P->num_sms, (nseg + nwarps - 1) / nwarps);
    kernel<<<grid, nwarps * 32, smem, st>>>(a, *tmap, sink, P->dev_error.p);
    GNNPRE_CUDA(cudaGetLastError());
    return GNNPRE_OK;
}

template <int G, int V, int U>
int launch_ceiling_shape(const SegArgs& a, float* sink, cudaStream_t st) {
    const unsigned grid = (unsigned)(((a.seg_hi - a.seg_lo) * G + kThreads - 1) / kThreads);
    k_ceiling<G, V, U><<<grid, kThreads, 0, st>>>(a, sink);
    GNNPRE_CUDA(cudaGetLastError());
    return GNNPRE_OK;
}

// The fetches of one hop over all column tiles of a slab, tiled and dispatched exactly as launch_segments does.
int launch_ceiling(const gnnpre_plan* P, const HopArgs& h, int64_t seg_lo, int64_t seg_hi, float* sink, cudaStream_t st) {
    if (seg_hi <= seg_lo) return GNNPRE_OK;
    const int32_t tile = segment_tile_width(P, h.width);
    for (int32_t f0 = 0; f0 < h.width; f0 += tile) {
        const int32_t w = std::min<int32_t>(tile, h.width - f0);
        SegArgs a{};
        a.segs = P->segments.p;
        a.seg_lo = seg_lo;
        a.seg_hi = seg_hi;
        a.colx = h.colx;
        a.colx_base = h.colx_edge_base;
        a.x = h.xprev + f0;
        a.ldx = h.ldx;
        a.f4 = w / 4;
        if (tile_uses_bulk_copy(P, w)) {
            if (a.f4 == 25) GNNPRE_TRY(launch_ceiling_tma<25>(P, a, sink, st));
            else if (a.f4 == 32) GNNPRE_TRY(launch_ceiling_tma<32>(P, a, sink, st));
            else GNNPRE_TRY(launch_ceiling_tma<0>(P, a, sink, st));
        } else if (a.f4 <= 4) GNNPRE_TRY((launch_ceiling_shape<4, 1, 4>(a, sink, st)));
        else if (a.f4 <= 8) GNNPRE_TRY((launch_ceiling_shape<8, 1, 8>(a, sink, st)));
        else if (a.f4 <= 16) GNNPRE_TRY((launch_ceiling_shape<16, 1, 8>(a, sink, st)));
        else if (a.f4 <= 32) GNNPRE_TRY((launch_ceiling_shape<32, 1, GNNPRE_SEG_U>(a, sink, st)));
        else if (a.f4 <= 64) GNNPRE_TRY((launch_ceiling_shape<32, 2, 4>(a, sink, st)));
        else GNNPRE_TRY((launch_ceiling_shape<32, 4, 2>(a, sink, st)));
    }
    return GNNPRE_OK;
}

}  // namespace

// Everything on the device: K hops, each a sweep over the column slabs and the edge blocks.
int propagate_resident(gnnpre_plan* P, const float* X, int64_t ldx, int32_t K, float* const* out, int64_t ldo,
                       cudaStream_t st, gnnpre_stats_t* stats, const WeightedSum* wsum) {
    // With stats, events bracket every hop and every launch of the segment kernel.
    std::vector<cudaEvent_t> hop_ev, seg_ev;
    auto mark = [&](std::vector<cudaEvent_t>& v) -> int {
        if (!stats) return GNNPRE_OK;
        cudaEvent_t e;
        GNNPRE_CUDA(cudaEventCreate(&e));
        v.push_back(e);
        GNNPRE_CUDA(cudaEventRecord(e, st));
        return GNNPRE_OK;
    };
    int64_t launches = 0, seg_launches = 0;
    int rc = mark(hop_ev);
    for (int32_t k = 0; k < K && rc == GNNPRE_OK; ++k) {
        const float* xprev = k == 0 ? X : out[k - 1];
        const int64_t ldp = k == 0 ? ldx : ldo;
        for (int32_t i = 0; i < P->c && rc == GNNPRE_OK; ++i) {
            const int64_t f_lo = (int64_t)i * P->slab_width;
            HopArgs h;
            h.colx = P->colx.p;
            h.colx_edge_base = 0;
            h.xprev = xprev + f_lo;
            h.x0 = X + f_lo;
            h.ldx0 = ldx;
            h.ldx = ldp;
            h.xout = out[k] + f_lo;
            h.ldo = ldo;
            h.width = (int32_t)std::min<int64_t>(P->slab_width, P->feat_dim - f_lo);
            if (wsum) {
                h.zsum = wsum->Z + f_lo;
                h.ldz = wsum->ldz;
                h.gamma = wsum->gamma[k + 1];
                h.gamma0 = wsum->gamma[0];
                h.zsum_first = k == 0;
            }
            const int tiles = (h.width + kMaxTile - 1) / kMaxTile;
            const int seg_tile = segment_tile_width(P, h.width);
            const int seg_tiles = (h.width + seg_tile - 1) / seg_tile;
            rc = launch_zero_empty_rows(P, h, st);
            launches += P->num_empty ? 1 : 0;
            const bool per_block = (P->flags & GNNPRE_FLAG_LAUNCH_PER_BLOCK) != 0;
            const size_t groups = per_block ? P->blocks.size() : 1;
            for (size_t j = 0; j < groups && rc == GNNPRE_OK; ++j) {
                const int64_t seg_lo = per_block ? P->blocks[j].seg_lo : 0;
                const int64_t seg_hi = per_block ? P->blocks[j].seg_hi : P->num_segments;
                const int64_t fix_lo = per_block ? P->blocks[j].fix_lo : 0;
                const int64_t fix_hi = per_block ? P->blocks[j].fix_hi : P->num_fixups;
                const int64_t hub_lo = per_block ? P->blocks[j].hub_lo : 0;
                const int64_t hub_hi = per_block ? P->blocks[j].hub_hi : P->num_hubs;
                if (seg_hi > seg_lo) {
                    rc = mark(seg_ev);
                    if (rc == GNNPRE_OK) rc = launch_segments(P, h, seg_lo, seg_hi, st);
                    if (rc == GNNPRE_OK) rc = mark(seg_ev);
                    launches += seg_tiles;
                    seg_launches += seg_tiles;
                }
                if (rc == GNNPRE_OK && fix_hi > fix_lo) {
                    rc = launch_fixups(P, h, fix_lo, fix_hi, hub_lo, hub_hi, st);
                    launches += tiles;
                }
            }
        }
        if (rc == GNNPRE_OK) rc = mark(hop_ev);
    }
    if (!P->last_use) GNNPRE_CUDA(cudaEventCreateWithFlags(&P->last_use, cudaEventDisableTiming));
    GNNPRE_CUDA(cudaEventRecord(P->last_use, st));  // the plan's scratch is in use until here
    if (stats) {
        if (rc == GNNPRE_OK && cudaStreamSynchronize(st) != cudaSuccess) rc = GNNPRE_ERR_CUDA;
        if (rc == GNNPRE_OK) rc = check_device_error(P);
        if (rc == GNNPRE_OK) {
            for (int32_t k = 0; k < K; ++k) cudaEventElapsedTime(&stats->hop_ms[k], hop_ev[(size_t)k], hop_ev[(size_t)k + 1]);
            cudaEventElapsedTime(&stats->total_ms, hop_ev[0], hop_ev[(size_t)K]);
            float seg_ms = 0.f;
            for (size_t j = 0; j + 1 < seg_ev.size(); j += 2) {
                float ms = 0.f;
                cudaEventElapsedTime(&ms, seg_ev[j], seg_ev[j + 1]);
                seg_ms += ms;
            }
            stats->segments_ms = seg_ms;
            stats->kernel_launches = launches;
            stats->segments_launches = seg_launches;
            stats->h2d_bytes = 0;
            stats->d2h_bytes = 0;
        }
        for (auto& e : hop_ev) cudaEventDestroy(e);
        for (auto& e : seg_ev) cudaEventDestroy(e);
    }
    return rc;
}

}  // namespace gnnpre

// Failure-detection self-tests: see include/gnnpre.h.
extern "C" int gnnpre_selftest_wait_timeout_async(gnnpre_plan_t* P, uint32_t polls, void* stream) {
    if (!P || !P->dev_error.p || polls == 0 || polls > 100000u) return GNNPRE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    gnnpre::k_wait_that_runs_out<<<1, 32, 0, st>>>(P->dev_error.p, polls);
    GNNPRE_CUDA(cudaGetLastError());
    return GNNPRE_OK;
}

extern "C" int gnnpre_selftest_wait_timeout(gnnpre_plan_t* P, uint32_t polls, void* stream) {
    GNNPRE_TRY(gnnpre_selftest_wait_timeout_async(P, polls, stream));
    return gnnpre_plan_status(P, stream);
}


// Measurement aid: see include/gnnpre.h.
extern "C" int gnnpre_gather_ceiling(gnnpre_plan_t* P, const float* X, int64_t ldx, float* sink, void* stream) {
    if (!P || !X || !sink) return GNNPRE_ERR_INVALID_ARG;
    if (P->structure_mem != GNNPRE_MEM_DEVICE) return GNNPRE_ERR_INVALID_ARG;
    if (ldx < P->feat_dim) return GNNPRE_ERR_INVALID_ARG;
    if (ldx % 4 != 0 || (reinterpret_cast<uintptr_t>(X) & 15u)) return GNNPRE_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (int32_t i = 0; i < P->c; ++i) {
        const int64_t f_lo = (int64_t)i * P->slab_width;
        gnnpre::HopArgs h;
        h.colx = P->colx.p;
        h.colx_edge_base = 0;
        h.xprev = X + f_lo;
        h.ldx = ldx;
        h.xout = nullptr;
        h.ldo = 0;
        h.x0 = nullptr;
        h.ldx0 = 0;
        h.width = (int32_t)std::min<int64_t>(P->slab_width, P->feat_dim - f_lo);
        GNNPRE_TRY(gnnpre::launch_ceiling(P, h, 0, P->num_segments, sink, st));
    }
    return GNNPRE_OK;
}
