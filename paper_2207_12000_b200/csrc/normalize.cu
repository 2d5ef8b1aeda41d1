// gnnpre_normalize: the normalised adjacency itself, edge block by edge block (Eq. 1 written block-wise
// as Eq. 10: S = sum_l D~^{-1/2} A~^(l) D~^{-1/2}).  The propagation path never needs these values (it
// applies the per-node scales on the fly); this export serves callers that want S as a matrix.
// Every value is evaluated in fp64 from the integer degrees and rounded once to fp32.
#include <algorithm>
#include <vector>

#include "gnnpre_internal.cuh"

namespace gnnpre {

namespace {

struct ValArgs {
    int64_t n;
    int64_t row_lo, row_hi;    // rows touched by this edge range (inclusive)
    int64_t e_lo, e_hi;        // edge range
    const int64_t* rowptr_t;
    const uint32_t* colx;      // entry of edge e at colx[e - colx_base]
    int64_t colx_base;
    const int32_t* deg;
    float* out;                // value of edge e goes to out[e - out_base]
    int64_t out_base;
    int op;
    double diag_weight;        // GIN: 1 + eps
};

// One warp per row of the range; lanes stride over the row's edges inside [e_lo, e_hi).
__global__ void k_edge_values(const ValArgs a) {
    const int64_t row = a.row_lo + (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (row > a.row_hi) return;
    const int64_t lo = max(a.rowptr_t[row], a.e_lo), hi = min(a.rowptr_t[row + 1], a.e_hi);
    const double di = (double)a.deg[row];
    for (int64_t e = lo + lane; e < hi; e += 32) {
        const int64_t col = (int64_t)(a.colx[e - a.colx_base] & ~kRowEndBit);
        double v;
        if (a.op == GNNPRE_OP_GCN_SYM) {
            v = (1.0 / sqrt(di + 1.0)) * (1.0 / sqrt((double)a.deg[col] + 1.0));
        } else if (a.op == GNNPRE_OP_SAGE_MEAN) {
            v = 1.0 / di;
        } else {
            v = col == row ? a.diag_weight : 1.0;
        }
        a.out[e - a.out_base] = (float)v;
    }
}

int launch_values(const ValArgs& a, cudaStream_t st) {
    if (a.e_hi <= a.e_lo) return GNNPRE_OK;
    const int64_t rows = a.row_hi - a.row_lo + 1;
    k_edge_values<<<(unsigned)((rows * 32 + 255) / 256), 256, 0, st>>>(a);
    GNNPRE_CUDA(cudaGetLastError());
    return GNNPRE_OK;
}

}  // namespace

}  // namespace gnnpre

using namespace gnnpre;

extern "C" int gnnpre_normalize(gnnpre_plan_t* P, float* vals_out, int32_t vals_mem, void* stream) {
    if (!P || !vals_out) return GNNPRE_ERR_INVALID_ARG;
    if (vals_mem != GNNPRE_MEM_DEVICE && vals_mem != GNNPRE_MEM_HOST) return GNNPRE_ERR_INVALID_ARG;
    if (P->nnz_tilde == 0) return GNNPRE_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ValArgs a;
    a.n = P->n;
    a.rowptr_t = P->rowptr_t.p;
    a.deg = P->deg.p;
    a.op = P->op;
    a.diag_weight = 1.0 + (double)P->gin_eps;
    const bool e_host = P->structure_mem == GNNPRE_MEM_HOST;
    if (!e_host && vals_mem == GNNPRE_MEM_DEVICE) {  // everything resident: all blocks in one launch
        a.row_lo = 0;
        a.row_hi = P->n - 1;
        a.e_lo = 0;
        a.e_hi = P->nnz_tilde;
        a.colx = P->colx.p;
        a.colx_base = 0;
        a.out = vals_out;
        a.out_base = 0;
        return launch_values(a, st);
    }
    // Block by block (the paper's a passes): E^(l) goes up on the plan's upload stream if it lives on the
    // host, the kernel runs on its compute stream, the values of block l go down on its download stream if
    // the caller wants them on the host.  Two buffers of each kind take turns and events order the three
    // streams, so block l+1 uploads and block l-1 downloads while block l computes.
    if (__sync_lock_test_and_set(&P->busy, 1)) return GNNPRE_ERR_BUSY;
    int64_t longest = 0;
    for (const Block& B : P->blocks) longest = std::max(longest, B.e_hi - B.e_lo);
    DevBuf<float> stage[2];
    std::vector<cudaEvent_t> events;
    auto record = [&](cudaStream_t s, cudaEvent_t* out) -> int {
        cudaEvent_t e = nullptr;
        GNNPRE_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        events.push_back(e);
        GNNPRE_CUDA(cudaEventRecord(e, s));
        *out = e;
        return GNNPRE_OK;
    };
    auto wait = [&](cudaStream_t s, cudaEvent_t e) -> int {
        if (e) GNNPRE_CUDA(cudaStreamWaitEvent(s, e, 0));
        return GNNPRE_OK;
    };
    auto body = [&]() -> int {
        GNNPRE_TRY(ensure_streams(P));
        if (vals_mem == GNNPRE_MEM_HOST) {
            GNNPRE_TRY(stage[0].alloc((size_t)longest));
            if (P->blocks.size() > 1) GNNPRE_TRY(stage[1].alloc((size_t)longest));
        }
        cudaEvent_t start = nullptr;
        GNNPRE_TRY(record(st, &start));
        GNNPRE_TRY(wait(P->s_h2d, start));
        GNNPRE_TRY(wait(P->s_compute, start));
        GNNPRE_TRY(wait(P->s_d2h, start));
        cudaEvent_t kernel_done[2] = {nullptr, nullptr};  // last kernel that read edge buffer sb / wrote value buffer sb
        cudaEvent_t drained[2] = {nullptr, nullptr};      // last download out of value buffer sb
        for (size_t j = 0; j < P->blocks.size(); ++j) {
            const Block& B = P->blocks[j];
            const int sb = (int)(j & 1);
            a.row_lo = B.row_lo;
            a.row_hi = B.row_hi;
            a.e_lo = B.e_lo;
            a.e_hi = B.e_hi;
            if (e_host) {
                if (P->stage_holds[sb] != (int64_t)j) {
                    GNNPRE_TRY(wait(P->s_h2d, kernel_done[sb]));
                    GNNPRE_CUDA(cudaMemcpyAsync(P->colx_stage[sb].p, P->colx_host.p + B.e_lo,
                                                sizeof(uint32_t) * (size_t)(B.e_hi - B.e_lo), cudaMemcpyHostToDevice,
                                                P->s_h2d));
                    P->stage_holds[sb] = (int64_t)j;
                    cudaEvent_t up = nullptr;
                    GNNPRE_TRY(record(P->s_h2d, &up));
                    GNNPRE_TRY(wait(P->s_compute, up));
                }
                a.colx = P->colx_stage[sb].p;
                a.colx_base = B.e_lo;
            } else {
                a.colx = P->colx.p;
                a.colx_base = 0;
            }
            if (vals_mem == GNNPRE_MEM_HOST) {
                GNNPRE_TRY(wait(P->s_compute, drained[sb]));
                a.out = stage[sb].p;
                a.out_base = B.e_lo;
            } else {
                a.out = vals_out;
                a.out_base = 0;
            }
            GNNPRE_TRY(launch_values(a, P->s_compute));
            GNNPRE_TRY(record(P->s_compute, &kernel_done[sb]));
            if (vals_mem == GNNPRE_MEM_HOST) {
                GNNPRE_TRY(wait(P->s_d2h, kernel_done[sb]));
                GNNPRE_CUDA(cudaMemcpyAsync(vals_out + B.e_lo, stage[sb].p, sizeof(float) * (size_t)(B.e_hi - B.e_lo),
                                            cudaMemcpyDeviceToHost, P->s_d2h));
                GNNPRE_TRY(record(P->s_d2h, &drained[sb]));
            }
        }
        return GNNPRE_OK;
    };
    int rc = body();
    // the staging buffers die with this call, and host results are promised on return
    for (cudaStream_t s : {P->s_h2d, P->s_compute, P->s_d2h})
        if (s && cudaStreamSynchronize(s) != cudaSuccess && rc == GNNPRE_OK) rc = GNNPRE_ERR_CUDA;
    for (cudaEvent_t e : events) cudaEventDestroy(e);
    if (rc != GNNPRE_OK) {
        (void)cudaGetLastError();
        P->stage_holds[0] = P->stage_holds[1] = -1;
    }
    __sync_lock_release(&P->busy);
    return rc;
}

// Eq. 11: least a with ceil((alpha_A B_A + alpha_S B_S) / a) + alpha_D B_D <= B_GPU (closed form).
extern "C" int gnnpre_solve_normalisation_blocks(int64_t B_A, int64_t B_S, int64_t B_D, int64_t alpha_A, int64_t alpha_S,
                                                 int64_t alpha_D, int64_t B_GPU, int64_t max_a, int64_t* a_out) {
    if (!a_out || B_A < 0 || B_S < 0 || B_D < 0 || alpha_A < 0 || alpha_S < 0 || alpha_D < 0 || max_a < 1)
        return GNNPRE_ERR_INVALID_ARG;
    const int64_t need = alpha_A * B_A + alpha_S * B_S;
    const int64_t room = B_GPU - alpha_D * B_D;
    if (room < 0 || (room == 0 && need > 0)) return GNNPRE_ERR_BUDGET_TOO_SMALL;
    const int64_t a = need == 0 ? 1 : (need + room - 1) / room;
    if (a > max_a) return GNNPRE_ERR_BUDGET_TOO_SMALL;
    *a_out = std::max<int64_t>(a, 1);
    return GNNPRE_OK;
}
