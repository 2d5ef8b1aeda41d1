// C-ABI glue: argument checks, status text, and the dispatch of gnnpre_propagate.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "gnnpre_internal.cuh"

namespace gnnpre {

namespace {
thread_local char g_last_error[512] = "";
// Allocations still allowed to succeed before one is reported as failed; negative = no injection.
std::atomic<int64_t> g_fail_countdown[2] = {{-1}, {-1}};

// Whether the [n, width] matrices at a (leading dimension lda floats) and b (ldb) share an element.  Column
// views of one wider buffer (equal leading dimensions, disjoint column ranges) do not.
bool matrices_overlap(const float* a, int64_t lda, const float* b, int64_t ldb, int64_t n, int64_t width) {
    if (n < 1 || width < 1) return false;
    const intptr_t pa = reinterpret_cast<intptr_t>(a), pb = reinterpret_cast<intptr_t>(b);
    const intptr_t span_a = ((n - 1) * lda + width) * (intptr_t)sizeof(float);
    const intptr_t span_b = ((n - 1) * ldb + width) * (intptr_t)sizeof(float);
    if (pa + span_a <= pb || pb + span_b <= pa) return false;  // the address ranges are disjoint
    if (lda != ldb) return true;                                // interleaved with different strides: assume they touch
    // same stride: element (i, p) of a meets (j, q) of b iff d = (i - j) * ld + (p - q), |p - q| < width
    const intptr_t diff = pb - pa;
    if (diff % (intptr_t)sizeof(float) != 0) return true;
    const intptr_t d = diff / (intptr_t)sizeof(float);
    intptr_t r = d % lda;
    if (r < 0) r += lda;
    return r < width || r > lda - width;
}
}  // namespace

bool injected_alloc_failure(int kind) {
    std::atomic<int64_t>& c = g_fail_countdown[kind];
    int64_t v = c.load();
    while (v >= 0) {
        if (c.compare_exchange_weak(v, v - 1)) return v == 0;  // the allocation that finds 0 fails; -1 = disarmed
    }
    return false;
}

void set_last_cuda_error(cudaError_t e, const char* what, const char* file, int line) {
    const char* base = std::strrchr(file, '/');
    std::snprintf(g_last_error, sizeof(g_last_error), "%s: %s (%s:%d)", cudaGetErrorName(e), what,
                  base ? base + 1 : file, line);
}

}  // namespace gnnpre

using namespace gnnpre;

extern "C" const char* gnnpre_last_cuda_error(void) { return g_last_error; }

extern "C" const char* gnnpre_status_string(int status) {
    switch (status) {
    case GNNPRE_OK: return "ok";
    case GNNPRE_ERR_INVALID_ARG: return "invalid argument";
    case GNNPRE_ERR_INVALID_CSR: return "CSR violates the input contract";
    case GNNPRE_ERR_ALIGN: return "misaligned pointer, leading dimension or feature width";
    case GNNPRE_ERR_OOM_DEVICE: return "out of device memory";
    case GNNPRE_ERR_OOM_HOST: return "out of host memory";
    case GNNPRE_ERR_BUDGET_TOO_SMALL: return "memory budget admits no (b, c)";
    case GNNPRE_ERR_CUDA: return "CUDA error";
    case GNNPRE_ERR_TIMEOUT: return "timed out";
    case GNNPRE_ERR_BUSY: return "plan is busy";
    case GNNPRE_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
    case GNNPRE_ERR_TOO_LARGE: return "problem exceeds the fixed scratch array of gnnpre_hop_static";
    default: return "unknown status";
    }
}

extern "C" int gnnpre_propagate(gnnpre_plan_t* P, const float* X, int64_t ldx, int32_t x_mem, int32_t K,
                                float* const* out, int64_t ldo, int32_t out_mem, void* stream, gnnpre_stats_t* stats) {
    if (!P || !X || !out || K < 1 || K > GNNPRE_MAX_HOPS) return GNNPRE_ERR_INVALID_ARG;
    if ((x_mem != GNNPRE_MEM_DEVICE && x_mem != GNNPRE_MEM_HOST) ||
        (out_mem != GNNPRE_MEM_DEVICE && out_mem != GNNPRE_MEM_HOST))
        return GNNPRE_ERR_INVALID_ARG;
    if (ldx < P->feat_dim || ldo < P->feat_dim) return GNNPRE_ERR_INVALID_ARG;
    if (ldx % 4 != 0 || ldo % 4 != 0 || (reinterpret_cast<uintptr_t>(X) & 15u)) return GNNPRE_ERR_ALIGN;
    for (int32_t k = 0; k < K; ++k) {
        if (!out[k]) return GNNPRE_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(out[k]) & 15u) return GNNPRE_ERR_ALIGN;
        // host and device addresses live in one address space (unified addressing), so one test serves both
        if (matrices_overlap(X, ldx, out[k], ldo, P->n, P->feat_dim)) return GNNPRE_ERR_INVALID_ARG;
        for (int32_t j = 0; j < k; ++j)
            if (matrices_overlap(out[j], ldo, out[k], ldo, P->n, P->feat_dim)) return GNNPRE_ERR_INVALID_ARG;
    }
    if (stats) std::memset(stats, 0, sizeof(*stats));
    int dev = -1;
    GNNPRE_CUDA(cudaGetDevice(&dev));
    if (dev != P->device) return GNNPRE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool resident = x_mem == GNNPRE_MEM_DEVICE && out_mem == GNNPRE_MEM_DEVICE && P->structure_mem == GNNPRE_MEM_DEVICE;
    const int rc = resident ? propagate_resident(P, X, ldx, K, out, ldo, st, stats)
                            : propagate_streamed(P, X, ldx, x_mem, K, out, ldo, out_mem, st, stats);
    // GNNPRE_LOG >= 1 in the environment: one line per call on stderr (2 adds the timeline of streamed calls)
    const char* log = std::getenv("GNNPRE_LOG");
    if (log && std::atoi(log) >= 1)
        std::fprintf(stderr, "[gnnpre] propagate n=%lld |E|=%lld F=%lld K=%d b=%d c=%d %s -> %s\n", (long long)P->n,
                     (long long)P->nnz_tilde, (long long)P->feat_dim, K, P->b, P->c,
                     resident ? "device-resident (enqueued)" : "streamed (complete)", gnnpre_status_string(rc));
    return rc;
}

extern "C" int gnnpre_propagate_weighted(gnnpre_plan_t* P, const float* X, int64_t ldx, int32_t K, float* const* out,
                                         int64_t ldo, const float* gamma, float* Z, int64_t ldz, void* stream) {
    if (!P || !X || !out || !gamma || !Z || K < 1 || K > GNNPRE_MAX_HOPS) return GNNPRE_ERR_INVALID_ARG;
    if (P->structure_mem != GNNPRE_MEM_DEVICE) return GNNPRE_ERR_INVALID_ARG;  // device-resident plans only
    if (ldx < P->feat_dim || ldo < P->feat_dim || ldz < P->feat_dim) return GNNPRE_ERR_INVALID_ARG;
    if (ldx % 4 != 0 || ldo % 4 != 0 || ldz % 4 != 0) return GNNPRE_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(X) & 15u) || (reinterpret_cast<uintptr_t>(Z) & 15u)) return GNNPRE_ERR_ALIGN;
    if (matrices_overlap(X, ldx, Z, ldz, P->n, P->feat_dim)) return GNNPRE_ERR_INVALID_ARG;
    for (int32_t k = 0; k < K; ++k) {
        if (!out[k]) return GNNPRE_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(out[k]) & 15u) return GNNPRE_ERR_ALIGN;
        if (matrices_overlap(X, ldx, out[k], ldo, P->n, P->feat_dim) ||
            matrices_overlap(Z, ldz, out[k], ldo, P->n, P->feat_dim))
            return GNNPRE_ERR_INVALID_ARG;
        // a hop may reuse the buffer of the hop before the previous one (two buffers suffice when only Z is wanted),
        // but never the one it reads
        if (k > 0 && matrices_overlap(out[k - 1], ldo, out[k], ldo, P->n, P->feat_dim)) return GNNPRE_ERR_INVALID_ARG;
    }
    int dev = -1;
    GNNPRE_CUDA(cudaGetDevice(&dev));
    if (dev != P->device) return GNNPRE_ERR_INVALID_ARG;
    WeightedSum w{gamma, Z, ldz};
    return propagate_resident(P, X, ldx, K, out, ldo, static_cast<cudaStream_t>(stream), nullptr, &w);
}

// See include/gnnpre.h.
extern "C" int gnnpre_plan_status(gnnpre_plan_t* P, void* stream) {
    if (!P) return GNNPRE_ERR_INVALID_ARG;
    GNNPRE_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    return check_device_error(P);
}

extern "C" int gnnpre_inject_alloc_failure(int64_t device_countdown, int64_t host_countdown) {
    g_fail_countdown[0].store(device_countdown < 0 ? -1 : device_countdown);
    g_fail_countdown[1].store(host_countdown < 0 ? -1 : host_countdown);
    return GNNPRE_OK;
}
