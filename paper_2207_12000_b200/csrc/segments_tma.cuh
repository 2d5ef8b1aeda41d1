// Segment kernel with the gathered rows staged through shared memory by the bulk-copy (TMA) engine.
// Included by propagate.cu inside its unnamed namespace (uses SegArgs, Segment, kRowEndBit).
//
// Why: the register kernel k_segments keeps at most (warps per SM) x 8 rows in flight, bounded by
// the register file and the load/store path; a gather of 400-512 B rows at random addresses needs on
// the order of 100 KB in flight per SM to hide HBM/L2 latency.  Here the copy engine moves the rows
// (completion counted in bytes on an mbarrier) and they wait in shared memory - kTmaStages x kTmaRows
// rows per warp, about 210 KB per SM - instead of registers.  The warp then sums the rows out of
// shared memory with conflict-free 128-bit reads.
//
// One CTA per SM, persistent: warp w of the grid walks segments w, w + W, w + 2W, ... (W = warps in
// the grid), so no atomics are involved and the summation order is the same as in k_segments
// (plain sums over steps of 8 edges, folded into the row's compensated sum): both kernels produce
// identical bits.
//
// Rows travel four at a time: one tile::gather4 tensor copy takes a column offset and four row
// indices of the [n, width] feature matrix (described by a tensor map whose box is one row high) and
// lands the four rows back to back in shared memory, so the copy engine is handed one instruction
// per four edges instead of one per edge (a plain cp.async.bulk per row was measured first: the
// engine is fed by one lane at a time, smsp__inst_executed_op_tma_ld equalled the edge count, and
// the issue loop dominated the instruction stream).  Groups of four rows start on 128-byte
// boundaries, as tensor copies require.
//
// Every wait on an mbarrier is bounded: after kTmaSpinLimit polls the warp records an error in
// a.error, drains what it has in flight (bounded as well) and leaves.
#pragma once

#ifndef GNNPRE_TMA_STAGES
#define GNNPRE_TMA_STAGES 2
#endif
#ifndef GNNPRE_TMA_ROWS
#define GNNPRE_TMA_ROWS 16
#endif
#ifndef GNNPRE_TMA_WARPS
#define GNNPRE_TMA_WARPS 16
#endif
constexpr int kTmaStages = GNNPRE_TMA_STAGES;  // chunks a warp keeps in flight
constexpr int kTmaRows = GNNPRE_TMA_ROWS;      // rows per stage = edges per chunk (8, 16 or 32)
constexpr int kTmaStep = 8;                    // edges per plain-sum step (same as k_segments' U for G = 32, V = 1)
constexpr int kTmaMaxWarps = GNNPRE_TMA_WARPS;
static_assert(kTmaRows % kTmaStep == 0 && kTmaRows % 4 == 0 && kTmaRows <= 32, "a chunk is a whole number of steps and fits one warp");
// A poll that finds the phase incomplete lets the hardware park the warp for up to kTmaSuspendNs
// before it returns, so waiting warps do not eat the issue slots of working ones; kTmaSpinLimit such
// polls (about two seconds at most) and the wait gives up.
constexpr uint32_t kTmaSuspendNs = 20000;
constexpr uint32_t kTmaSpinLimit = 100000;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// true once the phase with the given parity has completed
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity), "r"(kTmaSuspendNs)
        : "memory");
    return done != 0;
}

// Bounded wait; false if the limit ran out.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kTmaSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// Four rows r0..r3 of the tensor described by `tmap` (box = [width, 1]), columns from x0 on, land at
// dst, dst + row bytes, ...  dst is 128-byte aligned, x0 * 4 a multiple of 16.
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap* tmap, int x0, int r0, int r1, int r2, int r3,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar), "r"(x0), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
        : "memory");
}

// A float4 handled as two packed pairs: Blackwell adds and multiplies two fp32 per instruction
// (add/fma .f32x2).  Each lane of each pair is an ordinary IEEE operation, so results equal the scalar
// code's bit for bit.
struct Quad {
    float2 lo, hi;
};

__device__ __forceinline__ Quad quad_zero() { return {make_float2(0.f, 0.f), make_float2(0.f, 0.f)}; }

__device__ __forceinline__ Quad quad_load(const unsigned char* p) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    return {make_float2(v.x, v.y), make_float2(v.z, v.w)};
}

__device__ __forceinline__ void quad_add(Quad& a, const Quad& x) {
    a.lo = __fadd2_rn(a.lo, x.lo);
    a.hi = __fadd2_rn(a.hi, x.hi);
}

__device__ __forceinline__ void quad_fma(Quad& a, float w, const Quad& x) {
    const float2 ww = make_float2(w, w);
    a.lo = __ffma2_rn(ww, x.lo, a.lo);
    a.hi = __ffma2_rn(ww, x.hi, a.hi);
}

// Compensated addition of x into (sum, comp), as kahan1 does per component: a - b is evaluated as
// fma(-1, b, a), which rounds the same.
__device__ __forceinline__ void kahan_pair(float2& sum, float2& comp, const float2& x) {
    const float2 neg = make_float2(-1.f, -1.f);
    const float2 y = __ffma2_rn(neg, comp, x);
    const float2 t = __fadd2_rn(sum, y);
    comp = __ffma2_rn(neg, y, __ffma2_rn(neg, sum, t));
    sum = t;
}

__device__ __forceinline__ void quad_kahan(Quad& sum, Quad& comp, const Quad& x) {
    kahan_pair(sum.lo, comp.lo, x.lo);
    kahan_pair(sum.hi, comp.hi, x.hi);
}

// Per-stage bookkeeping a warp keeps in registers between issuing a chunk and summing it.
struct TmaChunk {
    uint32_t c;      // this lane's column entry (row-end mark in bit 31); 0 on padding lanes
    unsigned ends;   // row-end marks of the chunk, bit t = edge t
    int cnt;         // edges in the chunk
    int row;         // row of this lane's edge (valid where it ends a row; everywhere for GIN)
    float r, w;      // row scale of that row; weight of this lane's edge
};

// F4C: the row width in float4 when known at compile time (shared-memory offsets become immediates), else 0.
template <int OP, bool HAS_EMPTY, int F4C, int EP>
__global__ void __launch_bounds__(kTmaMaxWarps * 32, 1)
    k_segments_tma(const SegArgs a, const __grid_constant__ CUtensorMap tmap, int* error) {
    constexpr unsigned kFull = 0xffffffffu;
    extern __shared__ __align__(128) unsigned char tma_smem[];
    __shared__ __align__(8) unsigned long long bars[kTmaMaxWarps][kTmaStages];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    const uint32_t rb = F4C ? 16u * F4C : 16u * (uint32_t)a.f4;  // bytes of one row of this column tile
    const uint32_t group_bytes = (4u * rb + 127u) & ~127u;  // four rows, padded to the next 128-byte boundary
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
    // Lanes beyond the row's width never store; they re-read the row's last float4, the address their
    // quarter-warp already reads (one broadcast), so they add no shared-memory wavefront.
    const bool on = lane < a.f4;
    const uint32_t lane_off = on ? 16u * lane : rb - 16u;
    const unsigned lt_mask = (1u << lane) - 1u;

    const int64_t W = (int64_t)gridDim.x * nwarps;
    for (int64_t s = a.seg_lo + (int64_t)blockIdx.x * nwarps + warp; s < a.seg_hi && !failed; s += W) {
        const Segment g = a.segs[s];
        const int64_t e_beg = g.start, e_end = a.segs[s + 1].start;
        const int nchunks = (int)((e_end - e_beg + kTmaRows - 1) / kTmaRows);
        int rank_issue = g.rank;
        // column entries of the chunk that will be issued next, fetched one chunk ahead
        uint32_t c_next = 0;
        if (lane < kTmaRows && e_beg + lane < e_end) c_next = a.colx[e_beg + lane - a.colx_base];
        const int slot_head = g.slot_head, slot_tail = g.slot_tail;
        bool head_pending = slot_head >= 0;
        bool open = false;
        Quad acc = quad_zero(), tot = quad_zero(), cmp = quad_zero();
        TmaChunk ch[kTmaStages];

        // ---- ask the copy engine for the rows of chunk k, into stage st
        auto issue = [&](int k, int st) {
            TmaChunk& m = ch[st];
            const int64_t e0 = e_beg + (int64_t)k * kTmaRows;
            const int64_t left = e_end - e0;
            m.cnt = left >= kTmaRows ? kTmaRows : (int)left;
            const uint32_t c = c_next;
            c_next = 0;
            if (lane < kTmaRows && e0 + kTmaRows + lane < e_end) c_next = a.colx[e0 + kTmaRows + lane - a.colx_base];
            m.c = c;
            m.ends = __ballot_sync(kFull, (c & kRowEndBit) != 0);
            int row = rank_issue + __popc(m.ends & lt_mask);
            m.r = 1.f;
            m.w = 1.f;
            if (c & kRowEndBit) {
                if (HAS_EMPTY) row = a.nzrows[row];
                if (OP != GNNPRE_OP_GIN_SUM) m.r = a.rscale[row];
            }
            if (OP == GNNPRE_OP_GCN_SYM) {
                m.w = a.cscale[c & ~kRowEndBit];
            } else if (OP == GNNPRE_OP_GIN_SUM) {
                m.w = (int)(c & ~kRowEndBit) == row ? a.diag_weight : 1.f;
            }
            m.row = row;
            rank_issue += __popc(m.ends);
            const uint32_t bar = bar0 + 8u * st;
            // lanes 0, 4, 8, ... each hand the engine the rows of their four edges (padding lanes hold row 0)
            const int r0 = (int)(c & ~kRowEndBit);
            const int r1 = __shfl_down_sync(kFull, r0, 1), r2 = __shfl_down_sync(kFull, r0, 2),
                      r3 = __shfl_down_sync(kFull, r0, 3);
            const uint32_t groups = (uint32_t)(m.cnt + 3) >> 2;
            if (lane == 0) mbar_arrive_expect_tx(bar, groups * 4u * rb);
            __syncwarp();
            if ((lane & 3) == 0 && lane < m.cnt)
                tma_gather4(smem0 + st * stage_bytes + (uint32_t)(lane >> 2) * group_bytes, &tmap, 0, r0, r1, r2, r3, bar);
            inflight[st] = true;
        };

        // ---- a finished row (or the head part of one) leaves the warp
        auto flush = [&](int t, const TmaChunk& m) {
            const int row = __shfl_sync(kFull, m.row, t);
            const float r = __shfl_sync(kFull, m.r, t);
            const bool partial = head_pending;  // the row began in an earlier segment: leave the sum for the fix-up
            head_pending = false;
            float* dst = partial ? a.scratch + (int64_t)slot_head * a.scratch_ld : a.out + (int64_t)row * a.ldo;
            quad_kahan(tot, cmp, acc);
            if (on) {
                const float4 sum = make_float4(tot.lo.x, tot.lo.y, tot.hi.x, tot.hi.y);
                reinterpret_cast<float4*>(dst)[lane] = partial ? sum : finish_row_piece<EP>(sum, r, a.tp, row, lane);
            }
            acc = tot = cmp = quad_zero();
        };

        // ---- sum the rows of the chunk held by stage st
        auto consume = [&](int st) {
            const TmaChunk& m = ch[st];
            if (!mbar_wait_bounded(bar0 + 8u * st, phase[st])) {
                failed = true;
                return;
            }
            phase[st] ^= 1u;
            inflight[st] = false;
            const unsigned char* base = my_smem + st * stage_bytes + lane_off;
            if (kTmaRows == 2 * kTmaStep && m.cnt == kTmaRows && m.ends == 0) {
                // A full chunk inside one row (most of a hub's chunks): its two steps are summed side by
                // side, four rows of each at a time, so that four independent chains of adds are in
                // flight instead of two.  Each step's sum is still the plain chain over its 8 rows and
                // the two sums still join the compensated sum in edge order: same bits as the loop below.
                Quad acc2 = quad_zero();
#pragma unroll
                for (int h = 0; h < kTmaStep; h += 4) {
                    Quad xa[4], xb[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        xa[u] = quad_load(base + ((h + u) >> 2) * group_bytes + ((h + u) & 3) * rb);
                        xb[u] = quad_load(base + ((kTmaStep + h + u) >> 2) * group_bytes + ((kTmaStep + h + u) & 3) * rb);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (OP == GNNPRE_OP_SAGE_MEAN) {
                            quad_add(acc, xa[u]);
                            quad_add(acc2, xb[u]);
                        } else {
                            quad_fma(acc, __shfl_sync(kFull, m.w, h + u), xa[u]);
                            quad_fma(acc2, __shfl_sync(kFull, m.w, kTmaStep + h + u), xb[u]);
                        }
                    }
                }
                quad_kahan(tot, cmp, acc);
                quad_kahan(tot, cmp, acc2);
                acc = quad_zero();
                open = true;
                __syncwarp();
                return;
            }
            for (int t0 = 0; t0 < m.cnt; t0 += kTmaStep) {
                Quad x[kTmaStep];
#pragma unroll
                for (int u = 0; u < kTmaStep; ++u)
                    x[u] = quad_load(base + ((t0 + u) >> 2) * group_bytes + ((t0 + u) & 3) * rb);
                const unsigned step_ends = (m.ends >> t0) & ((1u << kTmaStep) - 1u);
                if (step_ends == 0 && t0 + kTmaStep <= m.cnt) {  // no row ends here: a straight run of adds
#pragma unroll
                    for (int u = 0; u < kTmaStep; ++u) {
                        if (OP == GNNPRE_OP_SAGE_MEAN) quad_add(acc, x[u]);
                        else quad_fma(acc, __shfl_sync(kFull, m.w, t0 + u), x[u]);
                    }
                } else {
#pragma unroll
                    for (int u = 0; u < kTmaStep; ++u) {
                        const int t = t0 + u;
                        if (t < m.cnt) {
                            if (OP == GNNPRE_OP_SAGE_MEAN) quad_add(acc, x[u]);
                            else quad_fma(acc, __shfl_sync(kFull, m.w, t), x[u]);
                            if ((m.ends >> t) & 1u) flush(t, m);
                        }
                    }
                }
                quad_kahan(tot, cmp, acc);  // this step's plain sum joins the row's compensated sum
                acc = quad_zero();
            }
            open = ((m.ends >> (m.cnt - 1)) & 1u) == 0;
            __syncwarp();  // every lane is done with the stage before it is refilled
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

        if (open) {  // the row holding the last edge continues in the next segment
            const int slot = head_pending ? slot_head : slot_tail;
            if (slot >= 0 && on)
                reinterpret_cast<float4*>(a.scratch + (int64_t)slot * a.scratch_ld)[lane] =
                    make_float4(tot.lo.x, tot.lo.y, tot.hi.x, tot.hi.y);
        }
    }

    if (failed) {
        // a wait ran out: report it, let the copies still in flight land (bounded), and leave
        if (lane == 0) atomicExch(error, 1);
#pragma unroll
        for (int st = 0; st < kTmaStages; ++st)
            if (inflight[st]) (void)mbar_wait_bounded(bar0 + 8u * st, phase[st]);
    }
}
