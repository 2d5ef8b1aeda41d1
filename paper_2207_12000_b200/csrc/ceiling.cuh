// Gather ceiling: the segment kernels with everything but the fetch and a plain row sum taken out.
// Included by propagate.cu inside its unnamed namespace (uses SegArgs, Segment, kRowEndBit and the
// bulk-copy helpers of segments_tma.cuh).
//
// For matrices that fit the L2 the HBM roofline says nothing about the segment kernels; what bounds them is
// how fast this device gathers rows of that width along that index stream.  These kernels measure it: they
// walk the same segments, read the same column entries and fetch the same rows through the same path
// (128-bit read-only loads into registers, or gather4 bulk copies into shared memory), add every fetched row
// into one plain running sum, and write four bytes per segment.  No scales, no row ends, no compensated
// sums, no output rows, no scratch.  Their results mean nothing; their duration is the yardstick.
#pragma once

template <int G, int V, int U>
__global__ void __launch_bounds__(kThreads, G <= 4 ? 4 : GNNPRE_SEG_MIN_BLOCKS) k_ceiling(const SegArgs a, float* __restrict__ sink) {
    constexpr unsigned kFull = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int gl = lane & (G - 1);
    const int64_t s = a.seg_lo + ((int64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    int64_t e = 0, e_end = 0;
    if (s < a.seg_hi) {
        e = a.segs[s].start;
        e_end = a.segs[s + 1].start;
    }
    const float4* xlane[V];
    const uint32_t ldx4 = (uint32_t)(a.ldx >> 2);
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int q = gl + v * G;
        xlane[v] = reinterpret_cast<const float4*>(a.x) + (q < a.f4 ? q : 0);
    }
    float4 acc[V];
#pragma unroll
    for (int v = 0; v < V; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    while (__any_sync(kFull, e < e_end)) {
        const int64_t left = e_end - e;
        const int cnt = left >= G ? G : (left > 0 ? (int)left : 0);
        uint32_t c = 0;  // lanes past the end fetch row 0
        if (gl < cnt) c = a.colx[e + gl - a.colx_base] & ~kRowEndBit;
        const int cnt_max = G == 32 ? cnt : __reduce_max_sync(kFull, cnt);
        for (int t0 = 0; t0 < cnt_max; t0 += U) {
            float4 x[U][V];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint64_t off = (uint64_t)__shfl_sync(kFull, c, t0 + u, G) * ldx4;
#pragma unroll
                for (int v = 0; v < V; ++v) x[u][v] = __ldg(xlane[v] + off);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    acc[v].x += x[u][v].x; acc[v].y += x[u][v].y;
                    acc[v].z += x[u][v].z; acc[v].w += x[u][v].w;
                }
            }
        }
        e += G;
    }
    float r = 0.f;
#pragma unroll
    for (int v = 0; v < V; ++v) r += (acc[v].x + acc[v].y) + (acc[v].z + acc[v].w);
    if (gl == 0 && s < a.seg_hi) sink[s] = r;
}

// The bulk-copy pipeline of k_segments_tma (same stages, same bounded waits, same give-up path) with the sums
// reduced to one plain chain per step pair.
template <int F4C>
__global__ void __launch_bounds__(kTmaMaxWarps * 32, 1)
    k_ceiling_tma(const SegArgs a, const __grid_constant__ CUtensorMap tmap, float* __restrict__ sink, int* error) {
    constexpr unsigned kFull = 0xffffffffu;
    extern __shared__ __align__(128) unsigned char tma_smem[];
    __shared__ __align__(8) unsigned long long bars[kTmaMaxWarps][kTmaStages];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    const uint32_t rb = F4C ? 16u * F4C : 16u * (uint32_t)a.f4;
    const uint32_t group_bytes = (4u * rb + 127u) & ~127u;
    const uint32_t stage_bytes = (kTmaRows / 4) * group_bytes;
    unsigned char* my_smem = tma_smem + (size_t)warp * kTmaStages * stage_bytes;
    const uint32_t smem0 = smem_u32(my_smem);
    const uint32_t bar0 = smem_u32(&bars[warp][0]);
    if (lane == 0) {
#pragma unroll
        for (int st = 0; st < kTmaStages; ++st) mbar_init(bar0 + 8u * st, 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    uint32_t phase[kTmaStages];
    bool inflight[kTmaStages];
#pragma unroll
    for (int st = 0; st < kTmaStages; ++st) {
        phase[st] = 0;
        inflight[st] = false;
    }
    bool failed = false;
    const uint32_t lane_off = lane < a.f4 ? 16u * lane : rb - 16u;

    const int64_t W = (int64_t)gridDim.x * nwarps;
    for (int64_t s = a.seg_lo + (int64_t)blockIdx.x * nwarps + warp; s < a.seg_hi && !failed; s += W) {
        const int64_t e_beg = a.segs[s].start, e_end = a.segs[s + 1].start;
        const int nchunks = (int)((e_end - e_beg + kTmaRows - 1) / kTmaRows);
        uint32_t c_next = 0;
        if (lane < kTmaRows && e_beg + lane < e_end) c_next = a.colx[e_beg + lane - a.colx_base];
        Quad acc = quad_zero(), acc2 = quad_zero();
        int cnt_of[kTmaStages];

        auto issue = [&](int k, int st) {
            const int64_t e0 = e_beg + (int64_t)k * kTmaRows;
            const int64_t left = e_end - e0;
            const int cnt = left >= kTmaRows ? kTmaRows : (int)left;
            cnt_of[st] = cnt;
            const uint32_t c = c_next;
            c_next = 0;
            if (lane < kTmaRows && e0 + kTmaRows + lane < e_end) c_next = a.colx[e0 + kTmaRows + lane - a.colx_base];
            const uint32_t bar = bar0 + 8u * st;
            const int r0 = (int)(c & ~kRowEndBit);
            const int r1 = __shfl_down_sync(kFull, r0, 1), r2 = __shfl_down_sync(kFull, r0, 2),
                      r3 = __shfl_down_sync(kFull, r0, 3);
            const uint32_t groups = (uint32_t)(cnt + 3) >> 2;
            if (lane == 0) mbar_arrive_expect_tx(bar, groups * 4u * rb);
            __syncwarp();
            if ((lane & 3) == 0 && lane < cnt)
                tma_gather4(smem0 + st * stage_bytes + (uint32_t)(lane >> 2) * group_bytes, &tmap, 0, r0, r1, r2, r3, bar);
            inflight[st] = true;
        };
        auto consume = [&](int st) {
            if (!mbar_wait_bounded(bar0 + 8u * st, phase[st])) {
                failed = true;
                return;
            }
            phase[st] ^= 1u;
            inflight[st] = false;
            const unsigned char* base = my_smem + st * stage_bytes + lane_off;
            const int groups = (cnt_of[st] + 3) >> 2;  // whole groups of four rows have landed (padding lanes fetched row 0)
            for (int gq = 0; gq < groups; gq += 2) {
                Quad xa[4], xb[4];
                const bool two = gq + 1 < groups;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    xa[u] = quad_load(base + gq * group_bytes + u * rb);
                    xb[u] = quad_load(base + (two ? gq + 1 : gq) * group_bytes + u * rb);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    quad_add(acc, xa[u]);
                    quad_add(acc2, xb[u]);
                }
            }
            __syncwarp();
        };
#pragma unroll
        for (int st = 0; st < kTmaStages; ++st)
            if (st < nchunks) issue(st, st);
        for (int k = 0; k < nchunks && !failed; k += kTmaStages) {
#pragma unroll
            for (int st = 0; st < kTmaStages; ++st) {
                if (k + st < nchunks && !failed) {
                    consume(st);
                    if (!failed && k + st + kTmaStages < nchunks) issue(k + st + kTmaStages, st);
                }
            }
        }
        if (failed) break;
        quad_add(acc, acc2);
        if (lane == 0) sink[s] = (acc.lo.x + acc.lo.y) + (acc.hi.x + acc.hi.y);
    }
    if (failed) {
        if (lane == 0) atomicExch(error, 1);
#pragma unroll
        for (int st = 0; st < kTmaStages; ++st)
            if (inflight[st]) (void)mbar_wait_bounded(bar0 + 8u * st, phase[st]);
    }
}
