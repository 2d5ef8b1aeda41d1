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
#include <algorithm>
#include <chrono>

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

struct SlabBuf {
    float* p = nullptr;
    cudaEvent_t kernel_read = nullptr;  // last kernel that reads it
    cudaEvent_t drained = nullptr;      // last device->host copy out of it
    cudaEvent_t filled = nullptr;       // the copy or kernels that fill it
};

int run(gnnpre_plan* P, const float* X, int64_t ldx, bool x_host, int32_t K, float* const* out, int64_t ldo,
        bool out_host, cudaStream_t user, gnnpre_stats_t* stats) {
    const int64_t n = P->n, w = P->slab_width;
    const bool e_host = P->structure_mem == GNNPRE_MEM_HOST;
    if (!P->s_h2d) GNNPRE_CUDA(cudaStreamCreateWithFlags(&P->s_h2d, cudaStreamNonBlocking));
    if (!P->s_d2h) GNNPRE_CUDA(cudaStreamCreateWithFlags(&P->s_d2h, cudaStreamNonBlocking));
    if (!P->s_compute) GNNPRE_CUDA(cudaStreamCreateWithFlags(&P->s_compute, cudaStreamNonBlocking));
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
    cudaEvent_t start = nullptr;
    GNNPRE_TRY(ev.record(user, &start));
    GNNPRE_TRY(wait(P->s_h2d, start));
    GNNPRE_TRY(wait(P->s_compute, start));
    GNNPRE_TRY(wait(P->s_d2h, start));

    int64_t h2d = 0, d2h = 0, launches = 0;
    cudaEvent_t stage_free[2] = {nullptr, nullptr};  // the kernels that last read each edge-block buffer
    int hop_turn = 0;

    auto upload_slab = [&](int32_t i) -> int {
        SlabBuf& b = in[i & 1];
        const int64_t f_lo = (int64_t)i * w, width = std::min<int64_t>(w, P->feat_dim - f_lo);
        GNNPRE_TRY(wait(P->s_h2d, b.kernel_read));
        GNNPRE_TRY(copy_rows(b.p, w, X + f_lo, ldx, width, n, cudaMemcpyHostToDevice, P->s_h2d));
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
                if (e_host) {
                    const int sb = (int)(j & 1);
                    if (P->stage_holds[sb] != (int64_t)j && B.e_hi > B.e_lo) {
                        GNNPRE_TRY(wait(P->s_h2d, stage_free[sb]));
                        GNNPRE_CUDA(cudaMemcpyAsync(P->colx_stage[sb].p, P->colx_host.p + B.e_lo,
                                                    sizeof(uint32_t) * (size_t)(B.e_hi - B.e_lo),
                                                    cudaMemcpyHostToDevice, P->s_h2d));
                        cudaEvent_t up = nullptr;
                        GNNPRE_TRY(ev.record(P->s_h2d, &up));
                        GNNPRE_TRY(wait(P->s_compute, up));
                        P->stage_holds[sb] = (int64_t)j;
                        h2d += 4 * (B.e_hi - B.e_lo);
                    }
                    h.colx = P->colx_stage[sb].p;
                    h.colx_edge_base = B.e_lo;
                }
                GNNPRE_TRY(launch_segments(P, h, B.seg_lo, B.seg_hi, P->s_compute));
                GNNPRE_TRY(launch_fixups(P, h, B.fix_lo, B.fix_hi, P->s_compute));
                launches += (B.seg_hi > B.seg_lo) + (B.fix_hi > B.fix_lo);
                cudaEvent_t done = nullptr;
                GNNPRE_TRY(ev.record(P->s_compute, &done));
                if (e_host) stage_free[j & 1] = done;
                if (out_host && B.done_row_hi > B.done_row_lo) {  // ship the rows this block completed
                    GNNPRE_TRY(wait(P->s_d2h, done));
                    const int64_t r0 = B.done_row_lo, rows = B.done_row_hi - B.done_row_lo;
                    GNNPRE_TRY(copy_rows(out[k] + r0 * ldo + f_lo, ldo, xout + r0 * ldd, ldd, width, rows,
                                         cudaMemcpyDeviceToHost, P->s_d2h));
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
    GNNPRE_CUDA(cudaStreamSynchronize(P->s_h2d));
    GNNPRE_CUDA(cudaStreamSynchronize(P->s_compute));
    GNNPRE_CUDA(cudaStreamSynchronize(P->s_d2h));
    GNNPRE_TRY(check_device_error(P));
    if (stats) {
        stats->h2d_bytes = h2d;
        stats->d2h_bytes = d2h;
        stats->kernel_launches = launches;
    }
    return GNNPRE_OK;
}

}  // namespace

int propagate_streamed(gnnpre_plan* P, const float* X, int64_t ldx, int32_t x_mem, int32_t K, float* const* out,
                       int64_t ldo, int32_t out_mem, cudaStream_t stream, gnnpre_stats_t* stats) {
    if (__sync_lock_test_and_set(&P->busy, 1)) return GNNPRE_ERR_BUSY;
    const auto t0 = std::chrono::steady_clock::now();
    int rc = run(P, X, ldx, x_mem == GNNPRE_MEM_HOST, K, out, ldo, out_mem == GNNPRE_MEM_HOST, stream, stats);
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
