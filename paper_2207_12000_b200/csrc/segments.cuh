// Register-gather segment kernel.  Included by propagate.cu inside its unnamed namespace (uses segments_common.cuh).
#pragma once

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
__global__ void __launch_bounds__(kThreads, G <= 4 ? 4 : GNNPRE_SEG_MIN_BLOCKS) k_segments(const SegArgs a) {
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
        if (cnt > 0) open = ((ends >> (cnt - 1)) & 1u) == 0;  // the chunk's last edge does not end its row
        const int cnt_max = G == 32 ? cnt : __reduce_max_sync(kFull, cnt);

        // ---- gather and accumulate, U rows in flight
        for (int t0 = 0; t0 < cnt_max; t0 += U) {
            float4 x[U][V];
            uint32_t craw[U];
            // Four-lane groups also hand every edge's row and row scale around ahead of time: with eight groups in a
            // warp a row ends somewhere in almost every step, and the two shuffles under a partial mask that a row end
            // otherwise costs are dearer than two plain ones per edge (measured: faster at G = 4, slower at G = 8, 16).
            constexpr bool kRowsAhead = G == 4;
            int rowv[U];
            float rv[U];
            float wv[U];  // the edges' weights, handed to the group together with their column entries (whole-warp
                          // shuffles outside any branch: a shuffle under a partial mask inside the per-edge
                          // condition below cost the weighted operators half again the time of the unweighted one)
#pragma unroll
            for (int u = 0; u < U; ++u) {
                craw[u] = __shfl_sync(kFull, c, t0 + u, G);
                if (OP != GNNPRE_OP_SAGE_MEAN) wv[u] = __shfl_sync(kFull, w, t0 + u, G);
                if (kRowsAhead) {
                    rowv[u] = __shfl_sync(kFull, my_row, t0 + u, G);
                    rv[u] = __shfl_sync(kFull, my_r, t0 + u, G);
                }
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
                        const float ww = wv[u];
#pragma unroll
                        for (int v = 0; v < V; ++v) {
                            acc[v].x = fmaf(ww, x[u][v].x, acc[v].x); acc[v].y = fmaf(ww, x[u][v].y, acc[v].y);
                            acc[v].z = fmaf(ww, x[u][v].z, acc[v].z); acc[v].w = fmaf(ww, x[u][v].w, acc[v].w);
                        }
                    }
                }
                if (craw[u] & kRowEndBit) {
                    // last edge of a row (never set on a padding lane): the whole group arrives here together
                    const int row = kRowsAhead ? rowv[u] : __shfl_sync(gmask, my_row, gshift + t);
                    const float r = kRowsAhead ? rv[u] : __shfl_sync(gmask, my_r, gshift + t);
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

