// Internal declarations shared by the library's translation units.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "gnnpre.h"

namespace gnnpre {

// ---------------------------------------------------------------- error plumbing
void set_last_cuda_error(cudaError_t e, const char* what, const char* file, int line);

#define GNNPRE_CUDA(call)                                                              \
    do {                                                                               \
        cudaError_t e__ = (call);                                                      \
        if (e__ != cudaSuccess) {                                                      \
            ::gnnpre::set_last_cuda_error(e__, #call, __FILE__, __LINE__);             \
            (void)cudaGetLastError();                                                  \
            return e__ == cudaErrorMemoryAllocation ? GNNPRE_ERR_OOM_DEVICE : GNNPRE_ERR_CUDA; \
        }                                                                              \
    } while (0)

#define GNNPRE_TRY(expr)                  \
    do {                                  \
        int s__ = (expr);                 \
        if (s__ != GNNPRE_OK) return s__; \
    } while (0)

// Failure injection for tests (gnnpre_inject_alloc_failure): true when this allocation must be
// reported as failed.  kind 0 = device memory, 1 = page-locked host memory.
bool injected_alloc_failure(int kind);

// Device allocation that frees itself.
template <typename T>
struct DevBuf {
    T* p = nullptr;
    size_t count = 0;
    DevBuf() = default;
    DevBuf(const DevBuf&) = delete;
    DevBuf& operator=(const DevBuf&) = delete;
    ~DevBuf() { reset(); }
    void reset() {
        if (p) cudaFree(p);
        p = nullptr;
        count = 0;
    }
    int alloc(size_t n) {
        reset();
        if (n == 0) return GNNPRE_OK;
        if (injected_alloc_failure(0)) {
            set_last_cuda_error(cudaErrorMemoryAllocation, "cudaMalloc (injected failure)", __FILE__, __LINE__);
            return GNNPRE_ERR_OOM_DEVICE;
        }
        GNNPRE_CUDA(cudaMalloc(reinterpret_cast<void**>(&p), n * sizeof(T)));
        count = n;
        return GNNPRE_OK;
    }
    size_t bytes() const { return count * sizeof(T); }
};

// Page-locked host allocation.
template <typename T>
struct PinnedBuf {
    T* p = nullptr;
    size_t count = 0;
    PinnedBuf() = default;
    PinnedBuf(const PinnedBuf&) = delete;
    PinnedBuf& operator=(const PinnedBuf&) = delete;
    ~PinnedBuf() { reset(); }
    void reset() {
        if (p) cudaFreeHost(p);
        p = nullptr;
        count = 0;
    }
    int alloc(size_t n) {
        reset();
        if (n == 0) return GNNPRE_OK;
        cudaError_t e = injected_alloc_failure(1) ? cudaErrorMemoryAllocation
                                                  : cudaMallocHost(reinterpret_cast<void**>(&p), n * sizeof(T));
        if (e != cudaSuccess) {
            set_last_cuda_error(e, "cudaMallocHost", __FILE__, __LINE__);
            (void)cudaGetLastError();
            return GNNPRE_ERR_OOM_HOST;
        }
        count = n;
        return GNNPRE_OK;
    }
    size_t bytes() const { return count * sizeof(T); }
};

// ---------------------------------------------------------------- the plan

// Bit 31 of an entry of the plan's column array marks the last edge of its row.
constexpr uint32_t kRowEndBit = 0x80000000u;

// One warp-level segment: edges [start, next segment's start).  A segment never crosses an
// edge-block boundary.  `rank` is the index, among rows that own at least one edge, of the row
// holding the segment's first edge.  slot_head >= 0: that row began in an earlier segment, and
// the part of it inside this segment goes to scratch row slot_head.  slot_tail >= 0: the row
// holding the last edge continues in the next segment and began in this one; its part goes to
// scratch row slot_tail.
struct Segment {
    int64_t start;
    int32_t rank;
    int32_t slot_head;
    int32_t slot_tail;
    int32_t pad;
};

// A row whose edges span segments seg_first..seg_last: its result is
// rscale[row] * (tail part of seg_first + head parts of seg_first+1 .. seg_last).  Those parts lie in
// consecutive scratch rows slot0, slot0 + 1, ... (the segments between the first and the last lie wholly
// inside the row, so each owns exactly one slot, and slots are numbered in segment order).
struct RowFixup {
    int32_t row;
    int32_t seg_first;
    int32_t seg_last;
    int32_t slot0;
};

struct Block {
    int64_t e_lo, e_hi;
    int32_t row_lo, row_hi;
    int32_t first_partial, last_partial;
    int64_t seg_lo, seg_hi;            // segments of this block
    int64_t fix_lo, fix_hi;            // fix-ups whose last segment lies in this block
    int64_t hub_lo, hub_hi;            // those among them with more than hub_parts parts (entries of `hubs`)
    int64_t done_row_lo, done_row_hi;  // rows complete once this block has run: [lo, hi)
};

}  // namespace gnnpre

struct gnnpre_plan {
    int device = 0;
    int64_t n = 0, nnz = 0, nnz_tilde = 0, feat_dim = 0;
    int32_t op = 0;
    float gin_eps = 0.f;
    float teleport_alpha = 0.f;
    int32_t b = 1, c = 1;
    int64_t slab_width = 0;
    int64_t B_S = 0, B_X = 0, B_fixed = 0, beta_S = 1, beta_X = 2, budget_bytes = 0;
    int32_t segment_edges = 0;
    uint32_t flags = 0;
    int32_t structure_mem = GNNPRE_MEM_DEVICE;
    bool rows_all_nonempty = true;  // every row owns an edge (always true with self-loops)
    int64_t num_nonempty = 0, num_empty = 0;

    // per-node arrays (device)
    gnnpre::DevBuf<int32_t> deg;
    gnnpre::DevBuf<float> rscale, cscale;
    gnnpre::DevBuf<int32_t> nzrows;     // rows owning >= 1 edge, ascending (only when !rows_all_nonempty)
    gnnpre::DevBuf<int32_t> emptyrows;  // rows owning no edge
    // support structure
    gnnpre::DevBuf<int64_t> rowptr_t;         // the support's row pointers
    gnnpre::DevBuf<uint32_t> colx;            // column | row-end bit, |E| entries (device-resident structure)
    gnnpre::PinnedBuf<uint32_t> colx_host;    // same, when the structure lives on the host
    gnnpre::DevBuf<uint32_t> colx_stage[2];   // double-buffered edge blocks (host structure)
    int64_t stage_holds[2] = {-1, -1};        // which block each staging buffer currently holds
    // decomposition
    std::vector<gnnpre::Block> blocks;
    gnnpre::DevBuf<gnnpre::Segment> segments;  // num_segments + 1 (the sentinel carries the end edge)
    gnnpre::DevBuf<gnnpre::RowFixup> fixups;
    gnnpre::DevBuf<int32_t> hubs;      // indices of the fix-ups with more than hub_parts parts, ascending
    int64_t num_hubs = 0;
    int32_t hub_parts = 0;
    int64_t num_segments = 0, num_fixups = 0, num_slots = 0;
    gnnpre::DevBuf<float> scratch;  // num_slots rows of slab_width floats
    gnnpre::DevBuf<int> dev_error;  // set by a kernel whose bounded wait ran out
    int num_sms = 0;
    // tensor maps of the matrices the bulk-copy kernel has been launched on (a cache: not part of the plan's meaning)
    struct TensorMapEntry {
        const float* x;
        int64_t ldx;
        int32_t f4;
        CUtensorMap map;
    };
    mutable std::vector<TensorMapEntry> tmaps;
    // streaming state
    gnnpre::DevBuf<float> slab[4];
    std::vector<gnnpre::DevBuf<float>> whole;  // panel schedule: X_0 .. X_K, each [n, feat_dim], grown on demand
    bool col_slabs_forced = false;             // c was given by the caller: the slab loop is then kept as asked
    cudaStream_t s_h2d = nullptr, s_d2h = nullptr, s_compute = nullptr, s_struct = nullptr;
    int busy = 0;
    // recorded on the caller's stream after the last work of every device-resident call: what
    // gnnpre_plan_destroy waits for instead of the whole device
    cudaEvent_t last_use = nullptr;

    ~gnnpre_plan();
    int64_t device_bytes() const;
    int64_t host_bytes() const;
};

namespace gnnpre {

// One launch's view of the operands.  All pointers are device pointers.
struct HopArgs {
    const uint32_t* colx;    // entry for absolute edge e is colx[e - colx_edge_base]
    int64_t colx_edge_base;
    const float* xprev;      // [n, ldx], already offset to the slab's first column
    int64_t ldx;
    float* xout;             // [n, ldo], likewise
    int64_t ldo;
    int32_t width;           // columns of this slab (multiple of 4)
    const float* x0;         // [n, ldx0] the slab of X_0, read only when the plan has a teleport term or zsum starts
    int64_t ldx0;
    // fixed-weight sum of hops, Z = gamma_0 X_0 + sum_k gamma_k X_k (nullptr = none): this hop adds gamma * X_k
    float* zsum = nullptr;   // [n, ldz], offset to the slab's first column
    int64_t ldz = 0;
    float gamma = 0.f;       // weight of the hop being computed
    float gamma0 = 0.f;      // weight of X_0
    bool zsum_first = false; // first hop: Z starts from gamma0 * X_0 instead of its old value
};

// propagate.cu
int launch_segments(const gnnpre_plan* plan, const HopArgs& a, int64_t seg_lo, int64_t seg_hi, cudaStream_t stream);
int launch_fixups(const gnnpre_plan* plan, const HopArgs& a, int64_t fix_lo, int64_t fix_hi, int64_t hub_lo, int64_t hub_hi,
                  cudaStream_t stream);
int launch_zero_empty_rows(const gnnpre_plan* plan, const HopArgs& a, cudaStream_t stream);
struct WeightedSum {         // optional extra output of propagate_resident
    const float* gamma;      // host, K + 1 weights
    float* Z;                // device [n, ldz]
    int64_t ldz;
};
int propagate_resident(gnnpre_plan* plan, const float* X, int64_t ldx, int32_t K, float* const* out, int64_t ldo,
                       cudaStream_t stream, gnnpre_stats_t* stats, const WeightedSum* wsum = nullptr);

// stream.cu
int ensure_streams(gnnpre_plan* plan);  // creates the plan's three side streams on first use
int propagate_streamed(gnnpre_plan* plan, const float* X, int64_t ldx, int32_t x_mem, int32_t K, float* const* out,
                       int64_t ldo, int32_t out_mem, cudaStream_t stream, gnnpre_stats_t* stats);

// plan.cu
int solve_budget(int64_t B_S, int64_t B_X, int64_t B_fixed, int64_t beta_S, int64_t beta_X, int64_t B_GPU,
                 int64_t max_b, int64_t max_c, int64_t* b_out, int64_t* c_out);
int check_device();
int check_device_error(gnnpre_plan* plan);  // synchronous read of plan->dev_error: GNNPRE_ERR_TIMEOUT if set
bool uses_bulk_copy(const gnnpre_plan* plan, int32_t width);

}  // namespace gnnpre
