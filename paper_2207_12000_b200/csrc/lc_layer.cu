// First dense stage of an LC model on a mini-batch of rows (Eq. 9 with the batch size and hidden
// width of the experimental settings): Y_k = act(X_k[batch] * W_1) for each precomputed hop X_k.
//
// This is the one dense contraction next to the aggregation path, so it runs on the 5th-generation
// tensor cores: a persistent, warp-specialised kernel with one CTA per SM.
//
//   warp 0   producer.  Per K-chunk of 32 features it gathers the 128 batch rows of the tile straight
//            out of the hop matrix with 32 tile::gather4 tensor copies (one per lane, four rows each,
//            128-byte swizzle) and fetches the matching [hidden, 32] chunk of the weight with one
//            tiled tensor copy; completion is counted in bytes on the stage's `full` mbarrier.
//   warp 1   one lane issues tcgen05.mma (kind::tf32, M = 128, N = hidden, K = 8 per instruction,
//            operands read from shared memory through swizzled K-major descriptors, fp32 accumulator
//            in tensor memory) and hands stages back with tcgen05.commit on the `empty` mbarrier.
//   warps 2-5  epilogue.  Each warp owns one quarter of the accumulator's 128 lanes, pulls it out of
//            tensor memory with tcgen05.ld, applies ReLU where asked and stores 64-byte pieces of its
//            row of Y.
//
// The accumulator is double-buffered (2 x 256 of the 512 tensor-memory columns), so the epilogue of
// one tile overlaps the copies and MMAs of the next.  The gathered rows never exist in HBM as a
// matrix of their own: the gather is the A-operand load.
//
// Arithmetic: the tensor core reads the fp32 operands as tf32 (it ignores the low 13 mantissa bits)
// and accumulates in fp32.
//
// Every wait is bounded.  A wait that runs out raises the CTA's abort flag and the caller's error
// word; every role then leaves its loop, the producer waits (bounded) for the copies it still has in
// flight, the MMA lane waits (bounded) for the tensor core to drain, and tensor memory is freed.
#include <algorithm>
#include <cstdint>

#include <cuda.h>

#include "gnnpre_internal.cuh"

namespace gnnpre {
namespace {

constexpr int kLcTileM = 128;                     // batch rows per tile = accumulator lanes
constexpr int kLcChunk = 32;                      // features per stage: 32 fp32 = one 128-byte swizzle row
constexpr int kLcStages = 4;
constexpr int kLcMaxHidden = 256;                 // N of one MMA, columns of one accumulator buffer
constexpr int kLcABytes = kLcTileM * 128;         // 16 KB
constexpr int kLcBBytes = kLcMaxHidden * 128;     // 32 KB
constexpr int kLcStageBytes = kLcABytes + kLcBBytes;
constexpr int kLcThreads = 192;
constexpr int kLcMaxHops = 8;                     // hop matrices (tensor maps) per launch
constexpr uint32_t kLcTmemCols = 512;
constexpr uint32_t kLcSuspendNs = 20000;          // a failed poll parks the warp for up to this long
constexpr uint32_t kLcSpinLimit = 50000;          // polls before a wait gives up (about a second)

struct LcMaps {
    CUtensorMap hop[kLcMaxHops];
    CUtensorMap w;
};

struct LcArgs {
    const int32_t* batch;  // row of the hop matrices for each batch position, or nullptr = identity
    int64_t batch_size;
    int32_t num_hops;
    int32_t tiles_m;       // ceil(batch_size / 128)
    int32_t k_chunks;      // ceil(F / 32)
    int32_t hidden;
    uint64_t relu_mask;    // bit k: apply ReLU to hop k's output
    float* y;
    int64_t ldy;
    int64_t y_hop_stride;
    int32_t* error;
};

__device__ __forceinline__ uint32_t lc_smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void lc_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void lc_mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void lc_mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool lc_mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity), "r"(kLcSuspendNs)
        : "memory");
    return done != 0;
}

// Bounded wait.  False when the limit ran out (the abort flag and the error word are then set) or
// when another role has already given up.
__device__ __forceinline__ bool lc_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* error) {
    for (uint32_t i = 0; i < kLcSpinLimit; ++i) {
        if (lc_mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    if (error) atomicExch(error, 1);
    return false;
}

__device__ __forceinline__ void lc_gather4(uint32_t dst, const CUtensorMap* tmap, int x0, int r0, int r1, int r2, int r3,
                                           uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar), "r"(x0), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
        : "memory");
}

__device__ __forceinline__ void lc_tile_load(uint32_t dst, const CUtensorMap* tmap, int x0, int y0, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar), "r"(x0), "r"(y0)
        : "memory");
}

// Shared-memory operand descriptor: K-major tile whose rows are 128 bytes (32 tf32) in the 128-byte
// swizzle, eight-row groups 1024 bytes apart.  `addr` is the tile's start (1024-byte aligned) plus
// 32 bytes per K-step of 8 inside the swizzle row.
__device__ __forceinline__ uint64_t lc_operand_desc(uint32_t addr) {
    uint64_t d = (uint64_t)((addr & 0x3ffffu) >> 4);   // start address, 16-byte units
    d |= (uint64_t)1 << 16;                             // leading-dimension offset: unused for this layout
    d |= (uint64_t)(1024 >> 4) << 32;                   // stride between eight-row groups
    d |= (uint64_t)1 << 46;                             // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                             // 128-byte swizzle
    return d;
}

// Instruction descriptor: fp32 accumulator, tf32 A and B, both K-major, M = 128, N = hidden.
__device__ __forceinline__ uint32_t lc_instr_desc(int n) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kLcTileM >> 4) << 24);
}

__device__ __forceinline__ void lc_mma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Makes the mbarrier track the completion of every MMA this thread has issued so far.
__device__ __forceinline__ void lc_mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void lc_tmem_load16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}

__global__ void __launch_bounds__(kLcThreads, 1) k_lc_first_layer(const __grid_constant__ LcMaps maps, const LcArgs a) {
    extern __shared__ unsigned char lc_smem[];
    __shared__ __align__(8) unsigned long long bars[2 * kLcStages + 5];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tiles0 = (lc_smem_u32(lc_smem) + 1023u) & ~1023u;  // operand tiles need 1024-byte alignment
    const uint32_t bar0 = lc_smem_u32(&bars[0]);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kLcStages + s); };
    auto acc_full_bar = [&](int b) { return bar0 + 8u * (2 * kLcStages + b); };
    auto acc_empty_bar = [&](int b) { return bar0 + 8u * (2 * kLcStages + 2 + b); };
    const uint32_t drain_bar = bar0 + 8u * (2 * kLcStages + 4);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kLcStages; ++s) {
            lc_mbar_init(full_bar(s), 1);
            lc_mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            lc_mbar_init(acc_full_bar(b), 1);
            lc_mbar_init(acc_empty_bar(b), 4);  // one arrival per epilogue warp
        }
        lc_mbar_init(drain_bar, 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(lc_smem_u32(&tmem_slot)),
                     "r"(kLcTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_slot;

    const int total_tiles = a.num_hops * a.tiles_m;
    const uint32_t stage_tx = (uint32_t)(kLcABytes + a.hidden * 128);

    if (warp == 0) {
        // ---------------------------------------------------------------- producer
        uint32_t g = 0;  // chunks issued so far, over all tiles
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const int hop = t / a.tiles_m, mt = t - hop * a.tiles_m;
            int r[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int64_t pos = (int64_t)mt * kLcTileM + 4 * lane + j;
                if (pos >= a.batch_size) pos = a.batch_size - 1;  // rows of a ragged last tile: fetched, never stored
                r[j] = a.batch ? __ldg(a.batch + pos) : (int)pos;
            }
            for (int kc = 0; kc < a.k_chunks; ++kc, ++g) {
                const int s = g % kLcStages;
                const uint32_t ph = (g / kLcStages) & 1u;
                if (!__all_sync(0xffffffffu, lc_wait(empty_bar(s), ph ^ 1u, abort_flag, a.error))) {
                    ok = false;
                    break;
                }
                const uint32_t a_dst = tiles0 + (uint32_t)s * kLcStageBytes;
                if (lane == 0) lc_mbar_arrive_expect_tx(full_bar(s), stage_tx);
                __syncwarp();
                lc_gather4(a_dst + 512u * lane, &maps.hop[hop], kc * kLcChunk, r[0], r[1], r[2], r[3], full_bar(s));
                if (lane == 0) lc_tile_load(a_dst + kLcABytes, &maps.w, kc * kLcChunk, 0, full_bar(s));
            }
        }
        // copies still in flight land in this CTA's shared memory: wait for them before leaving
        const uint32_t issued = g;
        for (int s = 0; s < kLcStages; ++s) {
            if (issued <= (uint32_t)s) continue;
            const uint32_t last = ((issued - 1 - s) / kLcStages) * kLcStages + s;  // last chunk that used stage s
            const uint32_t ph = (last / kLcStages) & 1u;
            for (uint32_t i = 0; i < kLcSpinLimit; ++i)
                if (lc_mbar_try_wait(full_bar(s), ph)) break;
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = lc_instr_desc(a.hidden);
            uint32_t g = 0;
            int it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
                const int buf = it & 1;
                const uint32_t acc_ph = (uint32_t)(it >> 1) & 1u;
                if (!lc_wait(acc_empty_bar(buf), acc_ph ^ 1u, abort_flag, a.error)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmem_d = tmem_base + (uint32_t)buf * kLcMaxHidden;
                for (int kc = 0; kc < a.k_chunks; ++kc, ++g) {
                    const int s = g % kLcStages;
                    const uint32_t ph = (g / kLcStages) & 1u;
                    if (!lc_wait(full_bar(s), ph, abort_flag, a.error)) {
                        ok = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_src = tiles0 + (uint32_t)s * kLcStageBytes;
                    const uint32_t b_src = a_src + kLcABytes;
#pragma unroll
                    for (int j = 0; j < kLcChunk / 8; ++j)
                        lc_mma_tf32(tmem_d, lc_operand_desc(a_src + 32u * j), lc_operand_desc(b_src + 32u * j), idesc,
                                    (kc | j) != 0);
                    lc_mma_commit(empty_bar(s));  // the stage is free once these MMAs have read it
                }
                if (ok) lc_mma_commit(acc_full_bar(buf));
            }
            // tensor memory may only be freed once the tensor core is idle
            lc_mma_commit(drain_bar);
            for (uint32_t i = 0; i < kLcSpinLimit; ++i)
                if (lc_mbar_try_wait(drain_bar, 0)) break;
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------------------- epilogue
        const int q = warp & 3;  // tensor-memory lanes 32q .. 32q+31 belong to this warp
        int it = 0;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, ++it) {
            const int hop = t / a.tiles_m, mt = t - hop * a.tiles_m;
            const int buf = it & 1;
            const uint32_t acc_ph = (uint32_t)(it >> 1) & 1u;
            if (!__all_sync(0xffffffffu, lc_wait(acc_full_bar(buf), acc_ph, abort_flag, a.error))) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int64_t pos = (int64_t)mt * kLcTileM + 32 * q + lane;
            const bool relu = (a.relu_mask >> hop) & 1u;
            float* yrow = a.y + (int64_t)hop * a.y_hop_stride + pos * a.ldy;
            const uint32_t taddr = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)buf * kLcMaxHidden;
            for (int c0 = 0; c0 < a.hidden; c0 += 16) {
                uint32_t v[16];
                lc_tmem_load16(taddr + (uint32_t)c0, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (pos < a.batch_size) {
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        float4 o = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]),
                                               __uint_as_float(v[j + 3]));
                        if (relu) {
                            o.x = fmaxf(o.x, 0.f);
                            o.y = fmaxf(o.y, 0.f);
                            o.z = fmaxf(o.z, 0.f);
                            o.w = fmaxf(o.w, 0.f);
                        }
                        *reinterpret_cast<float4*>(yrow + c0 + j) = o;
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) lc_mbar_arrive(acc_empty_bar(buf));
        }
        __syncwarp();
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kLcTmemCols) : "memory");
    }
}

int encode_map_2d(const float* base, int64_t inner, int64_t outer, int64_t ld, int box_inner, int box_outer,
                  CUtensorMap* out) {
    typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static encode_fn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        GNNPRE_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (q != cudaDriverEntryPointSuccess || !fn) return GNNPRE_ERR_CUDA;
        encode = reinterpret_cast<encode_fn>(fn);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    const cuuint32_t elem[2] = {1u, 1u};
    // elements outside the matrix (the ragged last K-chunk) are filled with zeros
    const CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, elem,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled", __FILE__, __LINE__);
        return GNNPRE_ERR_CUDA;
    }
    return GNNPRE_OK;
}

}  // namespace
}  // namespace gnnpre

using namespace gnnpre;

extern "C" int gnnpre_lc_first_layer(const float* const* hops, int32_t num_hops, int64_t n, int64_t feat_dim, int64_t ldh,
                                     const int32_t* batch, int64_t batch_size, const float* Wt, int64_t hidden, int64_t ldw,
                                     uint64_t relu_mask, float* Y, int64_t ldy, int64_t y_hop_stride, int32_t* error_flag,
                                     void* stream) {
    if (!hops || num_hops < 1 || num_hops > GNNPRE_MAX_HOPS || !Wt || (!Y && batch_size != 0)) return GNNPRE_ERR_INVALID_ARG;
    if (n < 1 || n > INT32_MAX || feat_dim < 1 || feat_dim > INT32_MAX - kLcChunk || batch_size < 0) return GNNPRE_ERR_INVALID_ARG;
    if (hidden < 16 || hidden > kLcMaxHidden || hidden % 16 != 0) return GNNPRE_ERR_INVALID_ARG;
    if (ldh < feat_dim || ldw < feat_dim || ldy < hidden) return GNNPRE_ERR_INVALID_ARG;
    if (!batch && batch_size > n) return GNNPRE_ERR_INVALID_ARG;
    if (ldh % 4 != 0 || ldw % 4 != 0 || ldy % 4 != 0 || y_hop_stride % 4 != 0) return GNNPRE_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(Wt) & 15u) || (reinterpret_cast<uintptr_t>(Y) & 15u)) return GNNPRE_ERR_ALIGN;
    for (int32_t k = 0; k < num_hops; ++k) {
        if (!hops[k]) return GNNPRE_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(hops[k]) & 15u) return GNNPRE_ERR_ALIGN;
    }
    const int64_t tiles_m = (batch_size + kLcTileM - 1) / kLcTileM;
    if (tiles_m * kLcMaxHops > INT32_MAX) return GNNPRE_ERR_INVALID_ARG;
    if (batch_size == 0) return GNNPRE_OK;

    int dev = -1, cc_major = 0, num_sms = 0;
    GNNPRE_CUDA(cudaGetDevice(&dev));
    GNNPRE_CUDA(cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev));
    if (cc_major != 10) return GNNPRE_ERR_UNSUPPORTED_ARCH;
    GNNPRE_CUDA(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev));
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    const size_t smem = (size_t)kLcStages * kLcStageBytes + 1024;
    GNNPRE_CUDA(cudaFuncSetAttribute(k_lc_first_layer, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));

    LcMaps maps;
    GNNPRE_TRY(encode_map_2d(Wt, feat_dim, hidden, ldw, kLcChunk, (int)hidden, &maps.w));
    for (int32_t k0 = 0; k0 < num_hops; k0 += kLcMaxHops) {  // at most kLcMaxHops tensor maps ride in one launch
        const int32_t kn = std::min<int32_t>(kLcMaxHops, num_hops - k0);
        for (int32_t k = 0; k < kLcMaxHops; ++k)
            GNNPRE_TRY(encode_map_2d(hops[k0 + std::min(k, kn - 1)], feat_dim, n, ldh, kLcChunk, 1, &maps.hop[k]));
        LcArgs a;
        a.batch = batch;
        a.batch_size = batch_size;
        a.num_hops = kn;
        a.tiles_m = (int32_t)tiles_m;
        a.k_chunks = (int32_t)((feat_dim + kLcChunk - 1) / kLcChunk);
        a.hidden = (int32_t)hidden;
        a.relu_mask = relu_mask >> k0;
        a.y = Y + (int64_t)k0 * y_hop_stride;
        a.ldy = ldy;
        a.y_hop_stride = y_hop_stride;
        a.error = error_flag;
        const int64_t total = (int64_t)kn * tiles_m;
        const unsigned grid = (unsigned)std::min<int64_t>(num_sms, total);
        k_lc_first_layer<<<grid, kLcThreads, smem, st>>>(maps, a);
        GNNPRE_CUDA(cudaGetLastError());
    }
    return GNNPRE_OK;
}
