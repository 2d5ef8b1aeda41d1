// What every propagation kernel shares: the epilogue of a finished row, the launch arguments, compensated addition.
// Included by propagate.cu inside its unnamed namespace, before the kernels.
#pragma once

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
constexpr int kMaxDevices = 64;

