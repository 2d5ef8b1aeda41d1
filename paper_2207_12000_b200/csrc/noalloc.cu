// gnnpre_hop_static: one hop  out = A^ X  straight from the caller's CSR, for callers that are not
// allowed to allocate device memory.  It is a simplified sibling of the segment kernel of
// propagate.cu: the edge list of A is cut into fixed-length segments, one warp walks one segment,
// rows cut by a segment boundary leave partial sums in scratch rows and a second kernel adds them
// up.  Here the scratch rows live in a fixed array inside the library's device image instead of a
// buffer obtained from cudaMalloc, nothing is precomputed (rows of edges are found by binary
// search, scale factors are recomputed from the row pointers), and the self-loop term is added
// when a row is finished.
#include <mutex>

#include "gnnpre_internal.cuh"

namespace gnnpre {

namespace {

constexpr size_t kStaticFloats = (size_t)GNNPRE_STATIC_SCRATCH_BYTES / sizeof(float);
constexpr int kMaxDevices = 64;
constexpr int kThreads = 256;
constexpr int kMaxV = 4;  // float4 per lane: rows of up to 512 floats

// Partial sums of cut rows: slot 2s is the head part of segment s (a row that began earlier),
// slot 2s + 1 its tail part (a row that goes on in the next segment).  Shared by every call on this
// device; a slot is always written by the segment kernel of a call before that call's fix-up kernel
// reads it, so nothing has to be cleared between calls.
static __device__ __align__(256) float g_static_scratch[kStaticFloats];

// Device addresses of g_static_scratch, one per device, filled on the first call on that device.
// (On the host the symbol's name is only a handle: the address a kernel can use comes from
// cudaGetSymbolAddress.)
float* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

int scratch_for_current_device(float** out) {
    int dev = -1;
    GNNPRE_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return GNNPRE_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        GNNPRE_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
        g_scratch_addr[dev] = static_cast<float*>(p);
    }
    *out = g_scratch_addr[dev];
    return GNNPRE_OK;
}

struct StaticArgs {
    int64_t n, nnz;
    const int64_t* rowptr;
    const int32_t* colidx;
    int op;
    float diag_weight;  // GIN: 1 + eps
    const float* x;
    int64_t ldx;
    float* out;
    int64_t ldo;
    int32_t f4;
    int32_t L;          // edges per segment
    int64_t nseg;
    float* scratch;
};

__device__ __forceinline__ void kahan_add(float4& s, float4& c, float w, const float4& x) {
    float y, t;
    y = fmaf(w, x.x, -c.x); t = s.x + y; c.x = (t - s.x) - y; s.x = t;
    y = fmaf(w, x.y, -c.y); t = s.y + y; c.y = (t - s.y) - y; s.y = t;
    y = fmaf(w, x.z, -c.z); t = s.z + y; c.z = (t - s.z) - y; s.z = t;
    y = fmaf(w, x.w, -c.w); t = s.w + y; c.w = (t - s.w) - y; s.w = t;
}

// Row holding edge e (0 <= e < nnz): the last i with rowptr[i] <= e.
__device__ __forceinline__ int64_t row_holding(const int64_t* __restrict__ rowptr, int64_t n, int64_t e) {
    int64_t lo = 0, hi = n;
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (rowptr[mid] <= e) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ float column_scale(const StaticArgs& a, int64_t j) {
    if (a.op != GNNPRE_OP_GCN_SYM) return 1.f;
    return (float)(1.0 / sqrt((double)(a.rowptr[j + 1] - a.rowptr[j]) + 1.0));
}

__device__ __forceinline__ float row_scale(const StaticArgs& a, int64_t i) {
    const int64_t d = a.rowptr[i + 1] - a.rowptr[i];
    if (a.op == GNNPRE_OP_GCN_SYM) return (float)(1.0 / sqrt((double)d + 1.0));
    if (a.op == GNNPRE_OP_SAGE_MEAN) return d > 0 ? (float)(1.0 / (double)d) : 0.f;
    return 1.f;
}

// Adds the self-loop term (if the operator has one), scales by r_i and stores row i.
__device__ __forceinline__ void finish_row(const StaticArgs& a, int64_t i, int lane, float4* tot, float4* cmp) {
    const float r = row_scale(a, i);
    const bool diag = a.op != GNNPRE_OP_SAGE_MEAN;
    const float wd = a.op == GNNPRE_OP_GCN_SYM ? r : a.diag_weight;
#pragma unroll
    for (int v = 0; v < kMaxV; ++v) {
        const int q = lane + 32 * v;
        if (q < a.f4) {
            if (diag) kahan_add(tot[v], cmp[v], wd, __ldg(reinterpret_cast<const float4*>(a.x + i * a.ldx) + q));
            float4 o = tot[v];
            o.x *= r; o.y *= r; o.z *= r; o.w *= r;
            reinterpret_cast<float4*>(a.out + i * a.ldo)[q] = o;
        }
    }
}

// One warp per segment of L edges of A.
__global__ void __launch_bounds__(kThreads) k_static_segments(const StaticArgs a) {
    constexpr unsigned kFull = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int64_t s = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    if (s >= a.nseg) return;
    const int64_t e_lo = s * a.L, e_hi = min(a.nnz, e_lo + (int64_t)a.L);
    int64_t r = row_holding(a.rowptr, a.n, e_lo);
    int64_t e = e_lo;
    while (e < e_hi) {
        const int64_t row_lo = a.rowptr[r], row_hi = a.rowptr[r + 1];
        const int64_t piece_hi = min(row_hi, e_hi);
        float4 tot[kMaxV], cmp[kMaxV];
#pragma unroll
        for (int v = 0; v < kMaxV; ++v) tot[v] = cmp[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int64_t base = e; base < piece_hi; base += 32) {
            const int cnt = (int)min((int64_t)32, piece_hi - base);
            int col = 0;
            float w = 0.f;
            if (lane < cnt) {
                col = a.colidx[base + lane];
                w = column_scale(a, col);
            }
            for (int t = 0; t < cnt; ++t) {
                const int cc = __shfl_sync(kFull, col, t);
                const float ww = __shfl_sync(kFull, w, t);
                const float4* src = reinterpret_cast<const float4*>(a.x + (int64_t)cc * a.ldx);
#pragma unroll
                for (int v = 0; v < kMaxV; ++v) {
                    const int q = lane + 32 * v;
                    if (q < a.f4) kahan_add(tot[v], cmp[v], ww, __ldg(src + q));
                }
            }
        }
        const bool began_earlier = row_lo < e_lo;
        const bool goes_on = row_hi > e_hi;
        if (!began_earlier && !goes_on) {
            finish_row(a, r, lane, tot, cmp);
        } else {
            float* dst = a.scratch + (2 * s + (began_earlier ? 0 : 1)) * (int64_t)(4 * a.f4);
#pragma unroll
            for (int v = 0; v < kMaxV; ++v) {
                const int q = lane + 32 * v;
                if (q < a.f4) reinterpret_cast<float4*>(dst)[q] = tot[v];
            }
        }
        e = piece_hi;
        if (e < e_hi) {  // next row that owns an edge (e < nnz, so one exists)
            ++r;
            while (a.rowptr[r + 1] == a.rowptr[r]) ++r;
        }
    }
}

// One warp per segment: if the row that began before this segment ends inside it, add up its parts.
__global__ void __launch_bounds__(kThreads) k_static_fixups(const StaticArgs a) {
    const int lane = threadIdx.x & 31;
    const int64_t s = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    if (s < 1 || s >= a.nseg) return;
    const int64_t e_lo = s * a.L, e_hi = min(a.nnz, e_lo + (int64_t)a.L);
    const int64_t r = row_holding(a.rowptr, a.n, e_lo);
    const int64_t row_lo = a.rowptr[r], row_hi = a.rowptr[r + 1];
    if (!(row_lo < e_lo && row_hi <= e_hi)) return;
    const int64_t s_first = row_lo / a.L;
    const int64_t stride = 4 * (int64_t)a.f4;
    float4 tot[kMaxV], cmp[kMaxV];
#pragma unroll
    for (int v = 0; v < kMaxV; ++v) tot[v] = cmp[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int64_t t = s_first; t <= s; ++t) {
        const float* src = a.scratch + (2 * t + (t == s_first ? 1 : 0)) * stride;
#pragma unroll
        for (int v = 0; v < kMaxV; ++v) {
            const int q = lane + 32 * v;
            if (q < a.f4) kahan_add(tot[v], cmp[v], 1.f, reinterpret_cast<const float4*>(src)[q]);
        }
    }
    finish_row(a, r, lane, tot, cmp);
}

// Rows without edges: the self-loop term alone, or zero.
__global__ void k_static_empty_rows(const StaticArgs a) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= a.n * a.f4) return;
    const int64_t i = t / a.f4;
    const int q = (int)(t % a.f4);
    if (a.rowptr[i + 1] != a.rowptr[i]) return;
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    if (a.op != GNNPRE_OP_SAGE_MEAN) {
        const float wd = a.op == GNNPRE_OP_GCN_SYM ? 1.f : a.diag_weight;  // D~ = 1: r * r = 1
        const float4 x = __ldg(reinterpret_cast<const float4*>(a.x + i * a.ldx) + q);
        o = make_float4(wd * x.x, wd * x.y, wd * x.z, wd * x.w);
    }
    reinterpret_cast<float4*>(a.out + i * a.ldo)[q] = o;
}

}  // namespace

}  // namespace gnnpre

using namespace gnnpre;

extern "C" int gnnpre_hop_static(const gnnpre_csr_t* csr, int32_t op, float gin_eps, int64_t feat_dim, const float* X,
                                 int64_t ldx, float* out, int64_t ldo, void* stream) {
    if (!csr || !X || !out || !csr->rowptr || (csr->nnz > 0 && !csr->colidx)) return GNNPRE_ERR_INVALID_ARG;
    if (csr->mem != GNNPRE_MEM_DEVICE) return GNNPRE_ERR_INVALID_ARG;
    if (csr->n < 1 || csr->n >= 0x7fffffffLL || csr->nnz < 0) return GNNPRE_ERR_INVALID_ARG;
    if (op < GNNPRE_OP_GCN_SYM || op > GNNPRE_OP_GIN_SUM) return GNNPRE_ERR_INVALID_ARG;
    if (feat_dim < 4 || ldx < feat_dim || ldo < feat_dim || out == X) return GNNPRE_ERR_INVALID_ARG;
    if (feat_dim % 4 != 0 || ldx % 4 != 0 || ldo % 4 != 0 || (reinterpret_cast<uintptr_t>(X) & 15u) ||
        (reinterpret_cast<uintptr_t>(out) & 15u))
        return GNNPRE_ERR_ALIGN;
    if (feat_dim > 128 * kMaxV) return GNNPRE_ERR_TOO_LARGE;
    GNNPRE_TRY(check_device());

    StaticArgs a;
    a.n = csr->n;
    a.nnz = csr->nnz;
    a.rowptr = csr->rowptr;
    a.colidx = csr->colidx;
    a.op = op;
    a.diag_weight = 1.0f + gin_eps;
    a.x = X;
    a.ldx = ldx;
    a.out = out;
    a.ldo = ldo;
    a.f4 = (int32_t)(feat_dim / 4);
    // the shortest segments, from 64 edges up, whose 2 scratch rows per segment fit the fixed array
    int64_t L = 64;
    while (L <= (1 << 20) && 2 * ((a.nnz + L - 1) / L) * feat_dim > (int64_t)kStaticFloats) L *= 2;
    if (L > (1 << 20)) return GNNPRE_ERR_TOO_LARGE;
    a.L = (int32_t)L;
    a.nseg = (a.nnz + L - 1) / L;
    GNNPRE_TRY(scratch_for_current_device(&a.scratch));

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t items = a.n * a.f4;
    k_static_empty_rows<<<(unsigned)((items + kThreads - 1) / kThreads), kThreads, 0, st>>>(a);
    GNNPRE_CUDA(cudaGetLastError());
    if (a.nseg > 0) {
        const unsigned grid = (unsigned)((a.nseg * 32 + kThreads - 1) / kThreads);
        k_static_segments<<<grid, kThreads, 0, st>>>(a);
        GNNPRE_CUDA(cudaGetLastError());
        if (a.nseg > 1) {
            k_static_fixups<<<grid, kThreads, 0, st>>>(a);
            GNNPRE_CUDA(cudaGetLastError());
        }
    }
    return GNNPRE_OK;
}
