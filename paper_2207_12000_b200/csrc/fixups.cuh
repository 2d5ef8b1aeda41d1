// Kernels that finish what the segment kernels leave: rows cut by segment boundaries, and rows without edges.
// Included by propagate.cu inside its unnamed namespace (uses Teleport, finish_row_piece, kahan4, kThreads).
#pragma once

struct FixArgs {
    const RowFixup* fix;
    int64_t fix_lo, fix_hi;
    const int32_t* hubs;     // fix-ups with more than hub_parts parts: entries [hub_lo, hub_hi) lie in [fix_lo, fix_hi)
    int64_t hub_lo, hub_hi;
    int32_t hub_parts;
    const float* scratch;
    int64_t scratch_ld;
    const float* rscale;
    float* out;
    int64_t ldo;
    int32_t f4;
    Teleport tp;
};

// (s, e) <- (s, e) + (t, f) for sums carried as value + error term: the values are added with the exact rounding
// error of that addition (branch-free two-sum) joining the error terms.  Symmetric in its operands.
__device__ __forceinline__ void pair_add1(float& s, float& e, float t, float f) {
    const float sum = s + t;
    const float bb = sum - s;
    const float lost = (s - (sum - bb)) + (t - bb);
    e = (e + f) + lost;
    s = sum;
}

__device__ __forceinline__ void pair_add4(float4& s, float4& e, const float4& t, const float4& f) {
    pair_add1(s.x, e.x, t.x, f.x);
    pair_add1(s.y, e.y, t.y, f.y);
    pair_add1(s.z, e.z, t.z, f.z);
    pair_add1(s.w, e.w, t.w, f.w);
}

// Adds up the parts of the cut rows.  A row's parts are P consecutive scratch rows; they are summed as a tree of
// fixed shape, so the result is the same from run to run, and - for tiles of up to 128 columns - the same whatever
// the tile width, so that a matrix cut into column tiles or slabs of any widths comes out bit-identical:
//   - chain c of C adds parts c, c + C, c + 2C, ... in that order with compensated additions, its loads issued
//     a batch ahead of its adds; the chains' sums (compensation folded in) then meet pairwise (c with c^1, then c^2,
//     then c^4), each carried as a value and an error term;
//   - an ordinary row gets one warp and C = 8 chains: a group of G lanes covers the row's width, so a warp holds
//     32 / G groups and every lane carries G / 4 chains (tiles wider than 128 columns, V > 1: one chain per warp);
//   - a hub row (P > hub_parts, listed by the plan) gets a whole CTA, C = 64 chains (8 per warp): the warps'
//     sums meet in shared memory and warp 0 adds them in warp order.
// The first (hub_hi - hub_lo) CTAs of the grid take the hubs, the others eight ordinary rows each.
template <int G, int V, int EP>
__global__ void __launch_bounds__(kThreads) k_row_fixups(const FixArgs a) {
    constexpr unsigned kFull = 0xffffffffu;
    constexpr int kWarps = kThreads / 32;
    constexpr int S = 32 / G;                  // lane groups per warp
    constexpr int CH = V == 1 ? G / 4 : 1;     // chains per lane
    constexpr int CW = S * CH;                 // chains per warp: 8, or 1 for wide tiles
    constexpr int kRounds = 16 / (CH * V);     // 16 float4 of parts in flight per lane
    __shared__ float4 meet[kWarps][2][G * V];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gl = lane & (G - 1), sub = lane / G;
    const int64_t nhub = a.hub_hi - a.hub_lo;
    const bool hub_cta = (int64_t)blockIdx.x < nhub;
    const int64_t i = hub_cta ? (int64_t)a.hubs[a.hub_lo + blockIdx.x]
                              : a.fix_lo + ((int64_t)blockIdx.x - nhub) * kWarps + warp;
    const int chains = hub_cta ? CW * kWarps : CW;           // chains that share the row
    const int chain0 = (hub_cta ? warp * CW : 0) + sub * CH;  // this lane's first chain
    int parts = 0, row = 0;
    const float* base = a.scratch;
    if (i < a.fix_hi) {
        const RowFixup f = a.fix[i];
        parts = f.seg_last - f.seg_first + 1;
        row = f.row;
        base += (int64_t)f.slot0 * a.scratch_ld;
    }
    const bool mine = i < a.fix_hi && (hub_cta || parts <= a.hub_parts);  // hubs are left to their CTAs
    if (!mine) parts = 0;
    bool on[V];
#pragma unroll
    for (int v = 0; v < V; ++v) on[v] = gl + v * G < a.f4;

    float4 acc[CH][V], cmp[CH][V];
#pragma unroll
    for (int j = 0; j < CH; ++j)
#pragma unroll
        for (int v = 0; v < V; ++v) acc[j][v] = cmp[j][v] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int p0 = 0; p0 < parts; p0 += chains * kRounds) {
        float4 part[kRounds][CH][V];
#pragma unroll
        for (int r = 0; r < kRounds; ++r) {
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                const int p = p0 + r * chains + chain0 + j;
                const float* src = base + (int64_t)(p < parts ? p : 0) * a.scratch_ld;
#pragma unroll
                for (int v = 0; v < V; ++v)
                    part[r][j][v] = p < parts && on[v] ? *reinterpret_cast<const float4*>(src + 4 * (gl + v * G))
                                                       : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int r = 0; r < kRounds; ++r) {
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                if (p0 + r * chains + chain0 + j < parts) {
#pragma unroll
                    for (int v = 0; v < V; ++v) kahan4(acc[j][v], cmp[j][v], part[r][j][v]);
                }
            }
        }
    }
    // The chains meet pairwise, first inside the lane (chains chain0 .. chain0 + CH - 1), then across the lane
    // groups of the warp.  A hub's partial sums can be far larger than their total (40,000 terms of either sign), so
    // every sum travels as a pair (value, error term) and each pairwise addition keeps its exact rounding error.
    float4 tot[V], err[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
#pragma unroll
        for (int j = 0; j < CH; ++j)  // a compensated sum stands for acc - cmp
            cmp[j][v] = make_float4(-cmp[j][v].x, -cmp[j][v].y, -cmp[j][v].z, -cmp[j][v].w);
#pragma unroll
        for (int step = 1; step < CH; step <<= 1) {
#pragma unroll
            for (int j = 0; j < CH; j += 2 * step) pair_add4(acc[j][v], cmp[j][v], acc[j + step][v], cmp[j + step][v]);
        }
        tot[v] = acc[0][v];
        err[v] = cmp[0][v];
#pragma unroll
        for (int off = G; off < 32; off <<= 1) {
            float4 os, oe;
            os.x = __shfl_xor_sync(kFull, tot[v].x, off); os.y = __shfl_xor_sync(kFull, tot[v].y, off);
            os.z = __shfl_xor_sync(kFull, tot[v].z, off); os.w = __shfl_xor_sync(kFull, tot[v].w, off);
            oe.x = __shfl_xor_sync(kFull, err[v].x, off); oe.y = __shfl_xor_sync(kFull, err[v].y, off);
            oe.z = __shfl_xor_sync(kFull, err[v].z, off); oe.w = __shfl_xor_sync(kFull, err[v].w, off);
            pair_add4(tot[v], err[v], os, oe);
        }
    }
    if (hub_cta) {  // uniform over the CTA
        if (sub == 0) {
#pragma unroll
            for (int v = 0; v < V; ++v) {
                meet[warp][0][gl + v * G] = tot[v];
                meet[warp][1][gl + v * G] = err[v];
            }
        }
        __syncthreads();
        if (warp != 0) return;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            tot[v] = meet[0][0][gl + v * G];
            err[v] = meet[0][1][gl + v * G];
            for (int w = 1; w < kWarps; ++w) pair_add4(tot[v], err[v], meet[w][0][gl + v * G], meet[w][1][gl + v * G]);
        }
    }
#pragma unroll
    for (int v = 0; v < V; ++v) {
        tot[v].x += err[v].x; tot[v].y += err[v].y; tot[v].z += err[v].z; tot[v].w += err[v].w;
    }
    if (mine && sub == 0) {
        const float r = a.rscale[row];
        float* dst = a.out + (int64_t)row * a.ldo;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int q = gl + v * G;
            if (on[v]) *reinterpret_cast<float4*>(dst + 4 * q) = finish_row_piece<EP>(tot[v], r, a.tp, row, q);
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

