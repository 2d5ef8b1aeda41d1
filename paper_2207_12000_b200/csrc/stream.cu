// Streaming pipeline for operands that live in host memory (the paper's setting: graph and features
// larger than the device, Section 3.2).  Algorithm 1's loops are kept, with the slab loop outermost
// so that a slab of X stays on the device for all K hops:
//
//   for slab i:   X_0[:, slab i]  host -> device                       (copy stream)
//     for hop k:  for block j:  E^(j) host -> device if E lives on the host (copy stream, double buffered)
//                               X_tmp[rows of block j] (+)= S^(j) X^(i)  (compute stream)
//                               rows finished by block j  device -> host (drain stream)
//
// Three streams and events between them overlap the two copy directions with the kernels.  Four
// slab buffers rotate: two take turns receiving X_0 slabs, two take turns as hop outputs (hop k
// reads one and writes the other while the drain stream empties the one written before).
//
// When the device has room for K + 1 whole matrices (on a 180 GB device it mostly has: the slabs are
// then needed for overlap, not for capacity) a second schedule keeps X_0 .. X_K whole on the device and
// moves COLUMN PANELS of unequal width instead (run_panels below): nothing can leave before the first
// slab of X has arrived, so the first slab is narrow (32 columns = 128-byte row pieces, the narrowest
// the host link still moves at ~85 % of full speed), the next ones double, and outputs leave in the
// widest pieces that are ready.  For F = 128, K = 2:
//
//   upload   X_0[:, 0:32)   X_0[:, 32:64)   X_0[:, 64:128)
//   compute  H1 0:32 | H1 32:64 | H2 0:64 | H1 64:128 | H2 64:128        (Hk = hop k on those columns)
//   drain    X_1[:, 0:32)   X_2[:, 0:64)   X_1[:, 32:128)   X_2[:, 64:128)
//
// Only 1/8 of the output bytes travel in 128-byte pieces and the link idles for a quarter of the time
// two equal slabs cost.
#include <algorithm>
#include <chrono>
#include <cstdio>
#include <cstdlib>

#include "gnnpre_internal.cuh"

namespace gnnpre {

namespace {

struct EventPool {
    std::vector<cudaEvent_t> all;
    ~EventPool() {
        for (auto e : all) cudaEventDestroy(e);
    }
    int record(cudaStream_t st, cudaEvent_t* out) {
        cudaEvent_t e;
        GNNPRE_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        all.push_back(e);
        GNNPRE_CUDA(cudaEventRecord(e, st));
        *out = e;
        return GNNPRE_OK;
    }
};

int wait(cudaStream_t st, cudaEvent_t e) {
    if (e) GNNPRE_CUDA(cudaStreamWaitEvent(st, e, 0));
    return GNNPRE_OK;
}

// rows x width floats between a strided and a dense matrix (or two strided ones)
int copy_rows(void* dst, int64_t dst_ld, const void* src, int64_t src_ld, int64_t width, int64_t rows,
              cudaMemcpyKind kind, cudaStream_t st) {
    if (rows <= 0 || width <= 0) return GNNPRE_OK;
    if (dst_ld == width && src_ld == width) {
        GNNPRE_CUDA(cudaMemcpyAsync(dst, src, sizeof(float) * (size_t)width * (size_t)rows, kind, st));
    } else {
        GNNPRE_CUDA(cudaMemcpy2DAsync(dst, sizeof(float) * (size_t)dst_ld, src, sizeof(float) * (size_t)src_ld,
                                      sizeof(float) * (size_t)width, (size_t)rows, kind, st));
    }
    return GNNPRE_OK;
}

// GNNPRE_LOG=2 in the environment: every copy and every block's kernels of a streamed call are bracketed by
// timing events and the timeline is printed to stderr when the call ends (milliseconds since the call began).
struct Trace {
    struct Span {
        char what[80];
        cudaEvent_t a, b;
    };
    std::vector<Span> spans;
    cudaEvent_t origin = nullptr;
    bool on = false;
    Trace() {
        const char* v = std::getenv("GNNPRE_LOG");
        on = v && std::atoi(v) >= 2;
    }
    ~Trace() {
        for (auto& s : spans) {
            cudaEventDestroy(s.a);
            cudaEventDestroy(s.b);
        }
        if (origin) cudaEventDestroy(origin);
    }
    void start(cudaStream_t user) {
        if (!on) return;
        if (cudaEventCreate(&origin) != cudaSuccess || cudaEventRecord(origin, user) != cudaSuccess) on = false;
    }
    // opens a span on `st`; close() records its end on the same stream
    int open(cudaStream_t st, const char* fmt, long long x = 0, long long y = 0, long long z = 0) {
        if (!on) return -1;
        Span sp;
        std::snprintf(sp.what, sizeof(sp.what), fmt, x, y, z);
        if (cudaEventCreate(&sp.a) != cudaSuccess) return -1;
        if (cudaEventCreate(&sp.b) != cudaSuccess) {
            cudaEventDestroy(sp.a);
            return -1;
        }
        cudaEventRecord(sp.a, st);
        spans.push_back(sp);
        return (int)spans.size() - 1;
    }
    void close(cudaStream_t st, int id) {
        if (id >= 0) cudaEventRecord(spans[(size_t)id].b, st);
    }
    void print() {  // after the streams have been synchronised
        if (!on) return;
        for (auto& s : spans) {
            float t0 = 0.f, t1 = 0.f;
            cudaEventElapsedTime(&t0, origin, s.a);
            cudaEventElapsedTime(&t1, origin, s.b);
            std::fprintf(stderr, "[gnnpre] %9.3f .. %9.3f ms  %s\n", t0, t1, s.what);
        }
    }
};

struct SlabBuf {
    float* p = nullptr;
    cudaEvent_t kernel_read = nullptr;  // last kernel that reads it
    cudaEvent_t drained = nullptr;      // last device->host copy out of it
    cudaEvent_t filled = nullptr;       // the copy or kernels that fill it
};

// Timing of the drain window for the statistics: call start, first output copy begins, last one has ended.
struct DrainTimer {
    cudaEvent_t start = nullptr, first = nullptr, last = nullptr;
    bool on = false;
    ~DrainTimer() {
        for (cudaEvent_t e : {start, first, last})
            if (e) cudaEventDestroy(e);
    }
    int begin(bool enabled, cudaStream_t user) {
        on = enabled;
        if (!on) return GNNPRE_OK;
        GNNPRE_CUDA(cudaEventCreate(&start));
        GNNPRE_CUDA(cudaEventCreate(&first));
        GNNPRE_CUDA(cudaEventCreate(&last));
        GNNPRE_CUDA(cudaEventRecord(start, user));
        return GNNPRE_OK;
    }
    bool seen_first = false;
    int before_copy(cudaStream_t s_d2h) {
        if (on && !seen_first) {
            seen_first = true;
            GNNPRE_CUDA(cudaEventRecord(first, s_d2h));
        }
        return GNNPRE_OK;
    }
    int finish(cudaStream_t s_d2h) {
        if (on && seen_first) GNNPRE_CUDA(cudaEventRecord(last, s_d2h));
        return GNNPRE_OK;
    }
    void report(gnnpre_stats_t* stats) {  // after the streams have been synchronised
        if (!on || !seen_first || !stats) return;
        cudaEventElapsedTime(&stats->startup_ms, start, first);
        cudaEventElapsedTime(&stats->drain_ms, first, last);
    }
};

// Edge block j on the device for the next launch: its column entries and their base edge.  With E on the
// host the block goes up through one of two staging buffers (on `up_stream`) unless it is still there.
struct BlockStager {
    gnnpre_plan* P;
    EventPool* ev;
    cudaStream_t up_stream;
    cudaEvent_t stage_free[2] = {nullptr, nullptr};  // the kernels that last read each staging buffer
    int64_t h2d = 0;
    int stage(size_t j, HopArgs* h) {
        const Block& B = P->blocks[j];
        if (P->structure_mem != GNNPRE_MEM_HOST) {
            h->colx = P->colx.p;
            h->colx_edge_base = 0;
            return GNNPRE_OK;
        }
        const int sb = (int)(j & 1);
        if (P->stage_holds[sb] != (int64_t)j && B.e_hi > B.e_lo) {
            GNNPRE_TRY(wait(up_stream, stage_free[sb]));
            GNNPRE_CUDA(cudaMemcpyAsync(P->colx_stage[sb].p, P->colx_host.p + B.e_lo,
                                        sizeof(uint32_t) * (size_t)(B.e_hi - B.e_lo), cudaMemcpyHostToDevice, up_stream));
            cudaEvent_t up = nullptr;
            GNNPRE_TRY(ev->record(up_stream, &up));
            GNNPRE_TRY(wait(P->s_compute, up));
            P->stage_holds[sb] = (int64_t)j;
            h2d += 4 * (B.e_hi - B.e_lo);
        }
        h->colx = P->colx_stage[sb].p;
        h->colx_edge_base = B.e_lo;
        return GNNPRE_OK;
    }
    void launched(size_t j, cudaEvent_t done) {
        if (P->structure_mem == GNNPRE_MEM_HOST) stage_free[j & 1] = done;
    }
};

int run_slabs(gnnpre_plan* P, const float* X, int64_t ldx, bool x_host, int32_t K, float* const* out, int64_t ldo,
              bool out_host, cudaStream_t user, gnnpre_stats_t* stats) {
    const int64_t n = P->n, w = P->slab_width;
    GNNPRE_TRY(ensure_streams(P));
    // slab buffers: 0, 1 receive X_0 slabs; 2, 3 are hop outputs
    if (x_host)
        for (int i = 0; i < 2; ++i)
            if (!P->slab[i].p) GNNPRE_TRY(P->slab[i].alloc((size_t)n * (size_t)w));
    if (out_host)
        for (int i = 2; i < 4; ++i)
            if (!P->slab[i].p) GNNPRE_TRY(P->slab[i].alloc((size_t)n * (size_t)w));
    SlabBuf in[2], hop[2];
    in[0].p = P->slab[0].p;
    in[1].p = P->slab[1].p;
    hop[0].p = P->slab[2].p;
    hop[1].p = P->slab[3].p;

    EventPool ev;
    DrainTimer timer;
    Trace trace;
    GNNPRE_TRY(timer.begin(stats != nullptr && out_host, user));
    trace.start(user);
    cudaEvent_t start = nullptr;
    GNNPRE_TRY(ev.record(user, &start));
    GNNPRE_TRY(wait(P->s_h2d, start));
    GNNPRE_TRY(wait(P->s_compute, start));
    GNNPRE_TRY(wait(P->s_d2h, start));

    int64_t h2d = 0, d2h = 0, launches = 0;
    BlockStager stager{P, &ev, P->s_h2d};
    int hop_turn = 0;

    auto upload_slab = [&](int32_t i) -> int {
        SlabBuf& b = in[i & 1];
        const int64_t f_lo = (int64_t)i * w, width = std::min<int64_t>(w, P->feat_dim - f_lo);
        GNNPRE_TRY(wait(P->s_h2d, b.kernel_read));
        const int span = trace.open(P->s_h2d, "h2d X[:, %lld:%lld)", f_lo, f_lo + width);
        GNNPRE_TRY(copy_rows(b.p, w, X + f_lo, ldx, width, n, cudaMemcpyHostToDevice, P->s_h2d));
        trace.close(P->s_h2d, span);
        GNNPRE_TRY(ev.record(P->s_h2d, &b.filled));
        h2d += 4 * width * n;
        return GNNPRE_OK;
    };

    if (x_host) GNNPRE_TRY(upload_slab(0));
    for (int32_t i = 0; i < P->c; ++i) {
        const int64_t f_lo = (int64_t)i * w, width = std::min<int64_t>(w, P->feat_dim - f_lo);
        const float* xprev = x_host ? in[i & 1].p : X + f_lo;
        int64_t ldp = x_host ? w : ldx;
        SlabBuf* prev_buf = x_host ? &in[i & 1] : nullptr;
        if (prev_buf) GNNPRE_TRY(wait(P->s_compute, prev_buf->filled));
        for (int32_t k = 0; k < K; ++k) {
            SlabBuf* dst_buf = out_host ? &hop[hop_turn & 1] : nullptr;
            if (out_host) ++hop_turn;
            float* xout = out_host ? dst_buf->p : out[k] + f_lo;
            const int64_t ldd = out_host ? w : ldo;
            if (dst_buf) {  // the buffer's earlier contents must have been read and drained
                GNNPRE_TRY(wait(P->s_compute, dst_buf->kernel_read));
                GNNPRE_TRY(wait(P->s_compute, dst_buf->drained));
            }
            HopArgs h;
            h.xprev = xprev;
            h.x0 = x_host ? in[i & 1].p : X + f_lo;  // the slab of X_0 stays put for all K hops
            h.ldx0 = x_host ? w : ldx;
            h.ldx = ldp;
            h.xout = xout;
            h.ldo = ldd;
            h.width = (int32_t)width;
            h.colx = P->colx.p;
            h.colx_edge_base = 0;
            GNNPRE_TRY(launch_zero_empty_rows(P, h, P->s_compute));
            launches += P->num_empty ? 1 : 0;
            for (size_t j = 0; j < P->blocks.size(); ++j) {
                const Block& B = P->blocks[j];
                GNNPRE_TRY(stager.stage(j, &h));
                GNNPRE_TRY(launch_segments(P, h, B.seg_lo, B.seg_hi, P->s_compute));
                GNNPRE_TRY(launch_fixups(P, h, B.fix_lo, B.fix_hi, B.hub_lo, B.hub_hi, P->s_compute));
                launches += (B.seg_hi > B.seg_lo) + (B.fix_hi > B.fix_lo);
                cudaEvent_t done = nullptr;
                GNNPRE_TRY(ev.record(P->s_compute, &done));
                stager.launched(j, done);
                if (out_host && B.done_row_hi > B.done_row_lo) {  // ship the rows this block completed
                    GNNPRE_TRY(wait(P->s_d2h, done));
                    GNNPRE_TRY(timer.before_copy(P->s_d2h));
                    const int64_t r0 = B.done_row_lo, rows = B.done_row_hi - B.done_row_lo;
                    const int dspan = j == 0 || j + 1 == P->blocks.size()
                                          ? trace.open(P->s_d2h, "d2h hop %lld cols %lld.. block %lld", k + 1, f_lo, (long long)j) : -1;
                    GNNPRE_TRY(copy_rows(out[k] + r0 * ldo + f_lo, ldo, xout + r0 * ldd, ldd, width, rows,
                                         cudaMemcpyDeviceToHost, P->s_d2h));
                    trace.close(P->s_d2h, dspan);
                    d2h += 4 * width * rows;
                }
                if (j + 1 == P->blocks.size()) {
                    if (x_host) in[i & 1].kernel_read = done;  // every hop may read X_0's slab (teleport term)
                    if (prev_buf) prev_buf->kernel_read = done;
                    if (dst_buf) {
                        dst_buf->filled = done;
                        if (out_host) GNNPRE_TRY(ev.record(P->s_d2h, &dst_buf->drained));
                    }
                }
            }
            // the next slab's X_0 is fetched while this slab's first hop runs
            if (k == 0 && x_host && i + 1 < P->c) GNNPRE_TRY(upload_slab(i + 1));
            xprev = xout;
            ldp = ldd;
            prev_buf = dst_buf;
        }
    }
    GNNPRE_TRY(timer.finish(P->s_d2h));
    GNNPRE_CUDA(cudaStreamSynchronize(P->s_h2d));
    GNNPRE_CUDA(cudaStreamSynchronize(P->s_compute));
    GNNPRE_CUDA(cudaStreamSynchronize(P->s_d2h));
    GNNPRE_TRY(check_device_error(P));
    if (stats) {
        stats->h2d_bytes = h2d + stager.h2d;
        stats->d2h_bytes = d2h;
        stats->kernel_launches = launches;
        stats->schedule = GNNPRE_SCHEDULE_SLABS;
        stats->upload_slabs = x_host ? P->c : 0;
        timer.report(stats);
    }
    trace.print();
    return GNNPRE_OK;
}

// ---------------------------------------------------------------- the panel schedule

struct Cols {
    int32_t lo, hi;
};

// Upload slabs of the panel schedule: 32, 32, then doubling (64, 128, ...), none wider than `cap`, the
// last one taking what is left.  F is a multiple of 32.
std::vector<Cols> panel_slabs(int32_t F, int32_t cap) {
    std::vector<Cols> v;
    int32_t lo = 0, w = 32;
    while (lo < F) {
        const int32_t width = std::min(std::min(w, cap), F - lo);
        v.push_back({lo, lo + width});
        lo += width;
        if (v.size() >= 2) w *= 2;
    }
    return v;
}

// One launch sequence of the compute stream: hop k on columns [lo, hi), all edge blocks; the rows each block
// completes then leave for the host as columns [drain_lo, drain_hi) of X_k (nothing if drain_hi <= drain_lo).
struct PanelJob {
    int32_t k, lo, hi;
    int32_t upload;  // index of the upload slab the job waits for, or -1
    int32_t drain_lo, drain_hi;
};

std::vector<PanelJob> panel_jobs(const std::vector<Cols>& s, int32_t K) {
    std::vector<PanelJob> jobs;
    const int32_t S = (int32_t)s.size();
    if (S == 1) {
        for (int32_t k = 1; k <= K; ++k) jobs.push_back({k, s[0].lo, s[0].hi, k == 1 ? 0 : -1, s[0].lo, s[0].hi});
        return jobs;
    }
    // the two narrow slabs: hop 1 apart (the first leaves at once, narrow; the second waits for the third slab and
    // leaves in one wide piece with it), the later hops on both together
    jobs.push_back({1, s[0].lo, s[0].hi, 0, s[0].lo, s[0].hi});
    if (S == 2) jobs.push_back({1, s[1].lo, s[1].hi, 1, s[1].lo, s[1].hi});
    else jobs.push_back({1, s[1].lo, s[1].hi, 1, 0, 0});
    for (int32_t k = 2; k <= K; ++k) jobs.push_back({k, s[0].lo, s[1].hi, -1, s[0].lo, s[1].hi});
    for (int32_t i = 2; i < S; ++i) {
        jobs.push_back({1, s[i].lo, s[i].hi, i, i == 2 ? s[1].lo : s[i].lo, s[i].hi});
        for (int32_t k = 2; k <= K; ++k) jobs.push_back({k, s[i].lo, s[i].hi, -1, s[i].lo, s[i].hi});
    }
    return jobs;
}

bool aligned128(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 127u) == 0; }

// Whether this call can run the panel schedule (see include/gnnpre.h, gnnpre_propagate).
bool panels_apply(const gnnpre_plan* P, const float* X, int64_t ldx, int32_t K, float* const* out, int64_t ldo) {
    const int64_t F = P->feat_dim;
    if (P->col_slabs_forced || P->c > 2 || F < 128 || F % 32 != 0 || P->slab_width < 64 || P->nnz_tilde == 0) return false;
    if ((ldx * 4) % 128 != 0 || (ldo * 4) % 128 != 0 || !aligned128(X)) return false;
    for (int32_t k = 0; k < K; ++k)
        if (!aligned128(out[k])) return false;
    int64_t held = P->device_bytes();
    for (const auto& w : P->whole) held -= (int64_t)w.bytes();
    const int64_t need = (int64_t)(K + 1) * P->n * F * (int64_t)sizeof(float);
    return held + need <= P->budget_bytes;
}

// GNNPRE_ERR_OOM_DEVICE (with the buffers released) when the device cannot hold the K + 1 matrices after all.
int ensure_whole_buffers(gnnpre_plan* P, int32_t K) {
    if (P->whole.size() < (size_t)K + 1) {
        std::vector<DevBuf<float>> grown((size_t)K + 1);
        for (size_t i = 0; i < P->whole.size(); ++i) std::swap(grown[i].p, P->whole[i].p), std::swap(grown[i].count, P->whole[i].count);
        P->whole.swap(grown);
    }
    for (int32_t k = 0; k <= K; ++k) {
        if (P->whole[(size_t)k].p) continue;
        const int rc = P->whole[(size_t)k].alloc((size_t)P->n * (size_t)P->feat_dim);
        if (rc != GNNPRE_OK) {
            for (auto& w : P->whole) w.reset();
            return rc;
        }
    }
    return GNNPRE_OK;
}

int run_panels(gnnpre_plan* P, const float* X, int64_t ldx, int32_t K, float* const* out, int64_t ldo, cudaStream_t user,
               gnnpre_stats_t* stats) {
    const int64_t n = P->n, F = P->feat_dim;
    GNNPRE_TRY(ensure_streams(P));
    if (!P->s_struct) GNNPRE_CUDA(cudaStreamCreateWithFlags(&P->s_struct, cudaStreamNonBlocking));
    const std::vector<Cols> slabs = panel_slabs((int32_t)F, (int32_t)P->slab_width);
    const std::vector<PanelJob> jobs = panel_jobs(slabs, K);

    EventPool ev;
    DrainTimer timer;
    Trace trace;
    GNNPRE_TRY(timer.begin(stats != nullptr, user));
    trace.start(user);
    cudaEvent_t start = nullptr;
    GNNPRE_TRY(ev.record(user, &start));
    for (cudaStream_t s : {P->s_h2d, P->s_compute, P->s_d2h, P->s_struct}) GNNPRE_TRY(wait(s, start));

    // X travels in slab order on its own stream; edge blocks (when E lives on the host) on another, so that a
    // block needed now never queues behind a slab needed later
    int64_t h2d = 0, d2h = 0, launches = 0;
    std::vector<cudaEvent_t> arrived(slabs.size(), nullptr);
    for (size_t i = 0; i < slabs.size(); ++i) {
        const int64_t width = slabs[i].hi - slabs[i].lo;
        const int span = trace.open(P->s_h2d, "h2d X[:, %lld:%lld)", slabs[i].lo, slabs[i].hi);
        GNNPRE_TRY(copy_rows(P->whole[0].p + slabs[i].lo, F, X + slabs[i].lo, ldx, width, n, cudaMemcpyHostToDevice, P->s_h2d));
        trace.close(P->s_h2d, span);
        GNNPRE_TRY(ev.record(P->s_h2d, &arrived[i]));
        h2d += 4 * width * n;
    }
    BlockStager stager{P, &ev, P->s_struct};
    for (const PanelJob& job : jobs) {
        if (job.upload >= 0) GNNPRE_TRY(wait(P->s_compute, arrived[(size_t)job.upload]));
        HopArgs h;
        h.xprev = P->whole[(size_t)job.k - 1].p + job.lo;
        h.ldx = F;
        h.x0 = P->whole[0].p + job.lo;  // read by the teleport term only
        h.ldx0 = F;
        h.xout = P->whole[(size_t)job.k].p + job.lo;
        h.ldo = F;
        h.width = job.hi - job.lo;
        h.colx = P->colx.p;
        h.colx_edge_base = 0;
        GNNPRE_TRY(launch_zero_empty_rows(P, h, P->s_compute));
        launches += P->num_empty ? 1 : 0;
        for (size_t j = 0; j < P->blocks.size(); ++j) {
            const Block& B = P->blocks[j];
            GNNPRE_TRY(stager.stage(j, &h));
            const int kspan = j == 0 || j + 1 == P->blocks.size()
                                  ? trace.open(P->s_compute, "hop %lld cols %lld.. block %lld", job.k, job.lo, (long long)j) : -1;
            GNNPRE_TRY(launch_segments(P, h, B.seg_lo, B.seg_hi, P->s_compute));
            GNNPRE_TRY(launch_fixups(P, h, B.fix_lo, B.fix_hi, B.hub_lo, B.hub_hi, P->s_compute));
            trace.close(P->s_compute, kspan);
            launches += (B.seg_hi > B.seg_lo) + (B.fix_hi > B.fix_lo);
            cudaEvent_t done = nullptr;
            GNNPRE_TRY(ev.record(P->s_compute, &done));
            stager.launched(j, done);
            if (job.drain_hi > job.drain_lo && B.done_row_hi > B.done_row_lo) {
                GNNPRE_TRY(wait(P->s_d2h, done));
                GNNPRE_TRY(timer.before_copy(P->s_d2h));
                const int64_t r0 = B.done_row_lo, rows = B.done_row_hi - B.done_row_lo, width = job.drain_hi - job.drain_lo;
                const int dspan = j == 0 || j + 1 == P->blocks.size()
                                      ? trace.open(P->s_d2h, "d2h hop %lld cols %lld.. block %lld", job.k, job.drain_lo, (long long)j) : -1;
                GNNPRE_TRY(copy_rows(out[job.k - 1] + r0 * ldo + job.drain_lo, ldo,
                                     P->whole[(size_t)job.k].p + r0 * F + job.drain_lo, F, width, rows,
                                     cudaMemcpyDeviceToHost, P->s_d2h));
                trace.close(P->s_d2h, dspan);
                d2h += 4 * width * rows;
            }
        }
    }
    GNNPRE_TRY(timer.finish(P->s_d2h));
    for (cudaStream_t s : {P->s_h2d, P->s_struct, P->s_compute, P->s_d2h}) GNNPRE_CUDA(cudaStreamSynchronize(s));
    GNNPRE_TRY(check_device_error(P));
    if (stats) {
        stats->h2d_bytes = h2d + stager.h2d;
        stats->d2h_bytes = d2h;
        stats->kernel_launches = launches;
        stats->schedule = GNNPRE_SCHEDULE_PANELS;
        stats->upload_slabs = (int32_t)slabs.size();
        timer.report(stats);
    }
    trace.print();
    return GNNPRE_OK;
}

}  // namespace

}  // namespace gnnpre

// Host only: see include/gnnpre.h.
extern "C" int gnnpre_describe_panels(int64_t feat_dim, int64_t slab_width, int32_t K, int32_t* jobs_out, int32_t max_jobs,
                                      int32_t* num_slabs_out, int32_t* num_jobs_out) {
    if (feat_dim < 32 || feat_dim % 32 != 0 || feat_dim > (1 << 20) || slab_width < 64 || K < 1 || K > GNNPRE_MAX_HOPS ||
        !num_slabs_out || !num_jobs_out || max_jobs < 0 || (max_jobs > 0 && !jobs_out))
        return GNNPRE_ERR_INVALID_ARG;
    const std::vector<gnnpre::Cols> slabs = gnnpre::panel_slabs((int32_t)feat_dim, (int32_t)std::min<int64_t>(slab_width, feat_dim));
    const std::vector<gnnpre::PanelJob> jobs = gnnpre::panel_jobs(slabs, K);
    *num_slabs_out = (int32_t)slabs.size();
    *num_jobs_out = (int32_t)jobs.size();
    for (size_t i = 0; i < jobs.size() && (int32_t)i < max_jobs; ++i) {
        const gnnpre::PanelJob& j = jobs[i];
        const int32_t rec[6] = {j.k, j.lo, j.hi, j.upload, j.drain_lo, j.drain_hi};
        for (int t = 0; t < 6; ++t) jobs_out[6 * i + t] = rec[t];
    }
    return GNNPRE_OK;
}

namespace gnnpre {

int ensure_streams(gnnpre_plan* P) {
    if (!P->s_h2d) GNNPRE_CUDA(cudaStreamCreateWithFlags(&P->s_h2d, cudaStreamNonBlocking));
    if (!P->s_d2h) GNNPRE_CUDA(cudaStreamCreateWithFlags(&P->s_d2h, cudaStreamNonBlocking));
    if (!P->s_compute) GNNPRE_CUDA(cudaStreamCreateWithFlags(&P->s_compute, cudaStreamNonBlocking));
    return GNNPRE_OK;
}

int propagate_streamed(gnnpre_plan* P, const float* X, int64_t ldx, int32_t x_mem, int32_t K, float* const* out,
                       int64_t ldo, int32_t out_mem, cudaStream_t stream, gnnpre_stats_t* stats) {
    if (__sync_lock_test_and_set(&P->busy, 1)) return GNNPRE_ERR_BUSY;
    const auto t0 = std::chrono::steady_clock::now();
    const bool x_host = x_mem == GNNPRE_MEM_HOST, out_host = out_mem == GNNPRE_MEM_HOST;
    int rc = GNNPRE_ERR_OOM_DEVICE;
    if (x_host && out_host && panels_apply(P, X, ldx, K, out, ldo)) {
        // the budget is a model: if the device turns out not to have the room, the slab schedule still runs
        rc = ensure_whole_buffers(P, K);
        if (rc == GNNPRE_OK) rc = run_panels(P, X, ldx, K, out, ldo, stream, stats);
        else if (rc == GNNPRE_ERR_OOM_DEVICE) rc = run_slabs(P, X, ldx, x_host, K, out, ldo, out_host, stream, stats);
    } else {
        for (auto& w : P->whole) w.reset();  // whole matrices kept from an earlier panel call give their room back
        rc = run_slabs(P, X, ldx, x_host, K, out, ldo, out_host, stream, stats);
    }
    if (rc != GNNPRE_OK) {
        // leave nothing in flight that still points at the caller's buffers
        cudaDeviceSynchronize();
        (void)cudaGetLastError();
        P->stage_holds[0] = P->stage_holds[1] = -1;
    }
    if (stats && rc == GNNPRE_OK)
        stats->total_ms = std::chrono::duration<float, std::milli>(std::chrono::steady_clock::now() - t0).count();
    __sync_lock_release(&P->busy);
    return rc;
}

}  // namespace gnnpre
