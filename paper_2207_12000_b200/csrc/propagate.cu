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

#include <cuda.h>

#include "gnnpre_internal.cuh"

namespace gnnpre {

namespace {

// The optional teleport term: a finished row r_i * sum becomes keep * (r_i * sum) + alpha * X_0[i].
struct Teleport {
    const float* x0;
    int64_t ldx0;
    float alpha, keep;  // keep = 1 - alpha
    // fixed-weight sum of hops (zsum == nullptr: none): Z += gamma * (the value stored for this hop)
    float* zsum;
    int64_t ldz;
    float gamma, gamma0;
    int zsum_first;
};

// EP, the epilogue of a finished row: 0 = scale only; 1 = scale and teleport term; 2 = the launch also accumulates the
// fixed-weight sum of hops (teleport decided at run time).  A compile-time switch, because the mere presence of the
// optional code slowed the plain kernels down although its branches were never taken (the L2-resident workload by
// 10 % for the teleport term and by 40 % for the sum).
constexpr int kEpPlain = 0, kEpTeleport = 1, kEpSum = 2;
template <int EP>
__device__ __forceinline__ float4 finish_row_piece(float4 sum, float scale, const Teleport& tp, int64_t row, int q) {
    float4 o = make_float4(sum.x * scale, sum.y * scale, sum.z * scale, sum.w * scale);
    if (EP == kEpTeleport || (EP == kEpSum && tp.alpha != 0.f)) {
        const float4 z = __ldg(reinterpret_cast<const float4*>(tp.x0 + row * tp.ldx0) + q);
        o.x = fmaf(tp.keep, o.x, tp.alpha * z.x);
        o.y = fmaf(tp.keep, o.y, tp.alpha * z.y);
        o.z = fmaf(tp.keep, o.z, tp.alpha * z.z);
        o.w = fmaf(tp.keep, o.w, tp.alpha * z.w);
    }
    if (EP == kEpSum) {  // every finished row piece passes here exactly once per hop
        float4* zp = reinterpret_cast<float4*>(tp.zsum + row * tp.ldz) + q;
        float4 acc;
        if (tp.zsum_first) {
            const float4 x = __ldg(reinterpret_cast<const float4*>(tp.x0 + row * tp.ldx0) + q);
            acc = make_float4(tp.gamma0 * x.x, tp.gamma0 * x.y, tp.gamma0 * x.z, tp.gamma0 * x.w);
        } else {
            acc = *zp;
        }
        acc.x = fmaf(tp.gamma, o.x, acc.x);
        acc.y = fmaf(tp.gamma, o.y, acc.y);
        acc.z = fmaf(tp.gamma, o.z, acc.z);
        acc.w = fmaf(tp.gamma, o.w, acc.w);
        *zp = acc;
    }
    return o;
}

// Which epilogue a launch needs.
inline int epilogue_of(const Teleport& tp) { return tp.zsum != nullptr ? kEpSum : tp.alpha != 0.f ? kEpTeleport : kEpPlain; }

struct SegArgs {
    const Segment* segs;
    int64_t seg_lo, seg_hi;
    const uint32_t* colx;
    int64_t colx_base;
    const float* x;
    int64_t ldx;
    float* out;
    int64_t ldo;
    float* scratch;
    int64_t scratch_ld;
    const float* rscale;
    const float* cscale;
    const int32_t* nzrows;
    int32_t f4;  // float4 per row of this column tile
    float diag_weight;  // GIN: 1 + eps
    Teleport tp;
};

// Compensated (Kahan) addition of x into the pair (sum, comp): the low-order bits that the addition
// drops are carried in comp.
__device__ __forceinline__ void kahan1(float& sum, float& comp, float x) {
    const float y = x - comp;
    const float t = sum + y;
    comp = (t - sum) - y;
    sum = t;
}

__device__ __forceinline__ void kahan4(float4& sum, float4& comp, const float4& x) {
    kahan1(sum.x, comp.x, x.x);
    kahan1(sum.y, comp.y, x.y);
    kahan1(sum.z, comp.z, x.z);
    kahan1(sum.w, comp.w, x.w);
}

constexpr int kThreads = 256;

// G lanes per segment, V float4 per lane (row width <= 4*G*V floats), U rows in flight per lane.
//
// Accumulation: the U rows of one step are added in a short plain fp32 chain, and that partial sum
// enters the row's running sum by a compensated (Kahan) addition, so the rounding error of a row
// stays at a few ulps of sum_j |w_j x_j| whatever its degree, at ~2 extra instructions per edge.
#ifndef GNNPRE_SEG_U
#define GNNPRE_SEG_U 8
#endif
#ifndef GNNPRE_SEG_MIN_BLOCKS
#define GNNPRE_SEG_MIN_BLOCKS 3
#endif
template <int G, int V, int U, int OP, bool HAS_EMPTY, int EP>
__global__ void __launch_bounds__(kThreads, GNNPRE_SEG_MIN_BLOCKS) k_segments(const SegArgs a) {
    constexpr unsigned kFull = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int gl = lane & (G - 1);
    const int gshift = lane & ~(G - 1);
    const unsigned glow = G == 32 ? kFull : ((1u << G) - 1u);
    const unsigned gmask = glow << gshift;
    const int64_t s = a.seg_lo + ((int64_t)blockIdx.x * kThreads + threadIdx.x) / G;

    int64_t e = 0, e_end = 0;
    int rank = 0, slot_head = -1, slot_tail = -1;
    if (s < a.seg_hi) {
        const Segment g = a.segs[s];
        e = g.start;
        e_end = a.segs[s + 1].start;
        rank = g.rank;
        slot_head = g.slot_head;
        slot_tail = g.slot_tail;
    }
    // Lane gl owns float4 columns gl, gl + G, ...; lanes beyond the row's width re-read column 0 so
    // that every load is unconditional and in bounds (their sums are never stored).
    bool on[V];
    const float4* xlane[V];
    const uint32_t ldx4 = (uint32_t)(a.ldx >> 2);
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int q = gl + v * G;
        on[v] = q < a.f4;
        xlane[v] = reinterpret_cast<const float4*>(a.x) + (on[v] ? q : 0);
    }
    bool head_pending = slot_head >= 0;  // the first row began in an earlier segment
    bool open = false;                   // the last edge seen so far did not end its row
    float4 acc[V], tot[V], cmp[V];       // this step's plain sum; the row's running sum and its compensation
#pragma unroll
    for (int v = 0; v < V; ++v) acc[v] = tot[v] = cmp[v] = make_float4(0.f, 0.f, 0.f, 0.f);

    while (__any_sync(kFull, e < e_end)) {
        // ---- this chunk's edges: lane gl of the group owns edge e + gl; lanes past the end hold 0,
        // a valid column without a row-end mark
        const int64_t left = e_end - e;
        const int cnt = left >= G ? G : (left > 0 ? (int)left : 0);
        uint32_t c = 0;
        if (gl < cnt) c = a.colx[e + gl - a.colx_base];
        const unsigned ends = (__ballot_sync(kFull, (c & kRowEndBit) != 0) >> gshift) & glow;
        int my_row = rank + __popc(ends & ((1u << gl) - 1u));
        float my_r = 1.f, w = 1.f;
        if (c & kRowEndBit) {
            if (HAS_EMPTY) my_row = a.nzrows[my_row];
            if (OP != GNNPRE_OP_GIN_SUM) my_r = a.rscale[my_row];
        }
        if (OP == GNNPRE_OP_GCN_SYM) {
            w = a.cscale[c & ~kRowEndBit];
        } else if (OP == GNNPRE_OP_GIN_SUM) {
            w = (int)(c & ~kRowEndBit) == my_row ? a.diag_weight : 1.f;  // every row owns its self-loop: rank == row
        }
        if (cnt > 0) open = (__shfl_sync(gmask, c, gshift + cnt - 1) & kRowEndBit) == 0;
        const int cnt_max = G == 32 ? cnt : __reduce_max_sync(kFull, cnt);

        // ---- gather and accumulate, U rows in flight
        for (int t0 = 0; t0 < cnt_max; t0 += U) {
            float4 x[U][V];
            uint32_t craw[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                craw[u] = __shfl_sync(kFull, c, t0 + u, G);
                const uint64_t off = (uint64_t)(craw[u] & ~kRowEndBit) * ldx4;
#pragma unroll
                for (int v = 0; v < V; ++v) x[u][v] = __ldg(xlane[v] + off);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int t = t0 + u;
                if (t < cnt) {
                    if (OP == GNNPRE_OP_SAGE_MEAN) {
#pragma unroll
                        for (int v = 0; v < V; ++v) {
                            acc[v].x += x[u][v].x; acc[v].y += x[u][v].y;
                            acc[v].z += x[u][v].z; acc[v].w += x[u][v].w;
                        }
                    } else {
                        const float ww = __shfl_sync(gmask, w, gshift + t);
#pragma unroll
                        for (int v = 0; v < V; ++v) {
                            acc[v].x = fmaf(ww, x[u][v].x, acc[v].x); acc[v].y = fmaf(ww, x[u][v].y, acc[v].y);
                            acc[v].z = fmaf(ww, x[u][v].z, acc[v].z); acc[v].w = fmaf(ww, x[u][v].w, acc[v].w);
                        }
                    }
                }
                if (craw[u] & kRowEndBit) {
                    // last edge of a row (never set on a padding lane): the whole group arrives here together
                    const int row = __shfl_sync(gmask, my_row, gshift + t);
                    const float r = __shfl_sync(gmask, my_r, gshift + t);
                    const bool partial = head_pending;  // the row began earlier: leave the sum for the fix-up
                    head_pending = false;
                    float* dst = partial ? a.scratch + (int64_t)slot_head * a.scratch_ld : a.out + (int64_t)row * a.ldo;
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        kahan4(tot[v], cmp[v], acc[v]);
                        if (on[v])
                            reinterpret_cast<float4*>(dst)[gl + v * G] =
                                partial ? tot[v] : finish_row_piece<EP>(tot[v], r, a.tp, row, gl + v * G);
                        acc[v] = tot[v] = cmp[v] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
            }
            if (t0 < cnt) {  // this step's plain sum joins the row's compensated sum (never on a padding
                             // step: the result must not depend on which segment shares the warp)
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    kahan4(tot[v], cmp[v], acc[v]);
                    acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
        rank += __popc(ends);
        e += G;
    }

    // ---- the row holding the last edge continues in the next segment
    if (open) {
        const int slot = head_pending ? slot_head : slot_tail;
        if (slot >= 0) {
            float* dst = a.scratch + (int64_t)slot * a.scratch_ld;
#pragma unroll
            for (int v = 0; v < V; ++v)
                if (on[v]) reinterpret_cast<float4*>(dst)[gl + v * G] = tot[v];
        }
    }
}

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

struct FixArgs {
    const RowFixup* fix;
    int64_t fix_lo, fix_hi;
    const Segment* segs;
    const float* scratch;
    int64_t scratch_ld;
    const float* rscale;
    float* out;
    int64_t ldo;
    int32_t f4;
    Teleport tp;
};

// One group per cut row: tail part of its first segment, then the head parts of the following ones,
// added in segment order.
template <int G, int V, int EP>
__global__ void __launch_bounds__(kThreads) k_row_fixups(const FixArgs a) {
    constexpr unsigned kFull = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int gl = lane & (G - 1);
    const int64_t i = a.fix_lo + ((int64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    int first = 0, last = -1, row = 0;
    if (i < a.fix_hi) {
        const RowFixup f = a.fix[i];
        first = f.seg_first;
        last = f.seg_last;
        row = f.row;
    }
    float4 acc[V], cmp[V];
#pragma unroll
    for (int v = 0; v < V; ++v) acc[v] = cmp[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    // A hub row spans hundreds of segments and its parts must be added in segment order, so the chain is bound by
    // load latency: the slot numbers of the next G segments are fetched while the current ones are added, and the
    // parts themselves are loaded kBatch at a time before they join the sum (the order of the additions is unchanged).
    constexpr int kBatch = 16 / V;  // 64 registers of parts in flight per lane
    auto slot_of = [&](int s0_) {
        int slot = -1;
        const int s = s0_ + gl;
        if (s <= last) slot = s == first ? a.segs[s].slot_tail : a.segs[s].slot_head;
        return slot;
    };
    int s0 = first;
    int slot = slot_of(s0);
    while (__any_sync(kFull, s0 <= last)) {
        const int cnt = last - s0 + 1 >= G ? G : (last >= s0 ? last - s0 + 1 : 0);
        const int slot_next = slot_of(s0 + G);
        const int cnt_max = G == 32 ? cnt : __reduce_max_sync(kFull, cnt);
        for (int t0 = 0; t0 < cnt_max; t0 += kBatch) {
            float4 part[kBatch][V];
            bool live[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int t = t0 + u;
                const int sl = __shfl_sync(kFull, slot, t & (G - 1), G);
                live[u] = t < cnt && sl >= 0;
                const float* p = a.scratch + (int64_t)(live[u] ? sl : 0) * a.scratch_ld;
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const int q = gl + v * G;
                    part[u][v] = live[u] && q < a.f4 ? *reinterpret_cast<const float4*>(p + 4 * q) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                if (live[u]) {
#pragma unroll
                    for (int v = 0; v < V; ++v)
                        if (gl + v * G < a.f4) kahan4(acc[v], cmp[v], part[u][v]);
                }
            }
        }
        s0 += G;
        slot = slot_next;
    }
    if (i < a.fix_hi) {
        const float r = a.rscale[row];
        float* dst = a.out + (int64_t)row * a.ldo;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int q = gl + v * G;
            if (q < a.f4) *reinterpret_cast<float4*>(dst + 4 * q) = finish_row_piece<EP>(acc[v], r, a.tp, row, q);
        }
    }
}

// Rows without any edge (SAGE, D_i = 0) are zero rows of the result.
// (With a teleport term they keep alpha * X_0[i].)
template <int EP>
__global__ void k_zero_rows(const int32_t* __restrict__ rows, int64_t count, float* __restrict__ out, int64_t ldo,
                            int32_t f4, const Teleport tp) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= count * f4) return;
    const int64_t r = rows[t / f4];
    const int q = (int)(t % f4);
    *reinterpret_cast<float4*>(out + r * ldo + 4 * q) = finish_row_piece<EP>(make_float4(0.f, 0.f, 0.f, 0.f), 0.f, tp, r, q);
}

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

// Bulk-copy variant: one persistent CTA per SM, as many warps as two stages of 32 rows each fit
// into the SM's shared memory (at most 8).
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
    static encode_fn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        GNNPRE_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (q != cudaDriverEntryPointSuccess || !fn) return GNNPRE_ERR_CUDA;
        encode = reinterpret_cast<encode_fn>(fn);
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

template <int OP, bool HAS_EMPTY, int F4C, int EP>
int launch_segments_tma_width(const gnnpre_plan* P, const SegArgs& a, cudaStream_t st) {
    const int nwarps = tma_warps(a.f4);
    const size_t smem = (size_t)nwarps * kTmaStages * tma_stage_bytes(a.f4);
    CUtensorMap tmap;
    GNNPRE_TRY(make_row_tensor_map(a.x, P->n, 4 * a.f4, a.ldx, &tmap));
    auto kernel = k_segments_tma<OP, HAS_EMPTY, F4C, EP>;
    GNNPRE_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int64_t nseg = a.seg_hi - a.seg_lo;
    const unsigned grid = (unsigned)std::min<int64_t>(P->num_sms, (nseg + nwarps - 1) / nwarps);
    kernel<<<grid, nwarps * 32, smem, st>>>(a, tmap, P->dev_error.p);
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
    const int64_t groups = a.fix_hi - a.fix_lo;
    const unsigned grid = (unsigned)((groups * G + kThreads - 1) / kThreads);
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

int launch_fixups(const gnnpre_plan* P, const HopArgs& h, int64_t fix_lo, int64_t fix_hi, cudaStream_t st) {
    if (fix_hi <= fix_lo) return GNNPRE_OK;
    for (int32_t f0 = 0; f0 < h.width; f0 += kMaxTile) {
        const int32_t w = std::min<int32_t>(kMaxTile, h.width - f0);
        FixArgs a;
        a.fix = P->fixups.p;
        a.fix_lo = fix_lo;
        a.fix_hi = fix_hi;
        a.segs = P->segments.p;
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
                if (seg_hi > seg_lo) {
                    rc = mark(seg_ev);
                    if (rc == GNNPRE_OK) rc = launch_segments(P, h, seg_lo, seg_hi, st);
                    if (rc == GNNPRE_OK) rc = mark(seg_ev);
                    launches += seg_tiles;
                    seg_launches += seg_tiles;
                }
                if (rc == GNNPRE_OK && fix_hi > fix_lo) {
                    rc = launch_fixups(P, h, fix_lo, fix_hi, st);
                    launches += tiles;
                }
            }
        }
        if (rc == GNNPRE_OK) rc = mark(hop_ev);
    }
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

// Failure-detection self-test: see include/gnnpre.h.
extern "C" int gnnpre_selftest_wait_timeout(gnnpre_plan_t* P, uint32_t polls, void* stream) {
    if (!P || !P->dev_error.p || polls == 0 || polls > 100000u) return GNNPRE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    gnnpre::k_wait_that_runs_out<<<1, 32, 0, st>>>(P->dev_error.p, polls);
    GNNPRE_CUDA(cudaGetLastError());
    GNNPRE_CUDA(cudaStreamSynchronize(st));
    return gnnpre::check_device_error(P);
}

