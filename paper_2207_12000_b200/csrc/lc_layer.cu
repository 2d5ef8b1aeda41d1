// First dense stage of an LC model on a mini-batch of rows (Eq. 9 with the batch size and hidden
// width of the experimental settings): Y_k = act(X_k[batch] * W_1) for each precomputed hop X_k.
//
// This is the one dense contraction next to the aggregation path, so it runs on the 5th-generation
// tensor cores: a persistent, warp-specialised kernel with one CTA per SM.
//
//   warps 0-3  producers.  Per K-chunk of 32 features they gather the 128 batch rows of the tile straight
//            out of the hop matrix into the 128-byte-swizzled operand layout with 16-byte asynchronous
//            copies (cp.async: no registers, zero fill past the last feature and for rows outside the
//            batch), keep three chunks in flight beyond the one they announce, and arrive on the stage's
//            `full` mbarrier after a proxy fence.  (Tensor copies in tile::gather4 mode were measured
//            first: at 128 bytes per gathered row the copy engine's per-row rate, about 95 rows per
//            microsecond and SM, capped the kernel at 60 % of what the output stores alone sustain.)
//            The weight travels by tiled tensor copies, counted in bytes on an mbarrier.
//   warp 4   one lane issues tcgen05.mma (kind::tf32, M = 128, N = hidden, K = 8 per instruction,
//            operands read from shared memory through swizzled K-major descriptors, fp32 accumulator
//            in tensor memory) and hands stages back with tcgen05.commit on the `empty` mbarrier.
//   warps 5-12  epilogue.  Two warps share each quarter of the accumulator's 128 lanes (even and odd
//            column boxes); a warp pulls its part out of tensor memory with tcgen05.ld 32 columns at a
//            time, applies ReLU where asked, lays the [32, 32] box down in shared memory (128-byte
//            swizzle, conflict-free) and hands it to the copy engine as a tensor store, which writes
//            whole lines and clips the ragged edges.
//
// A weight of up to 128 KB is loaded once per CTA and stays in shared memory; a larger one is
// streamed chunk by chunk beside the rows.
// The accumulator is double-buffered (2 x 256 of the 512 tensor-memory columns), so the epilogue of
// one tile overlaps the copies and MMAs of the next.  The gathered rows never exist in HBM as a
// matrix of their own: the gather is the A-operand load.
//
// Arithmetic: the tensor core reads the fp32 operands as tf32 (8 exponent bits, 10 explicit mantissa
// bits; the low 13 bits are cut, not rounded: a relative error below 2^-10 per operand) and accumulates in fp32.  k_lc_first_layer_x3 below
// feeds every operand as two tf32 numbers instead.
//
// Every wait is bounded.  A wait that runs out raises the CTA's abort flag and the caller's error
// word; every role then leaves its loop, the producers wait for the copies they still have in
// flight, the MMA lane waits (bounded) for the tensor core to drain, and tensor memory is freed.
#include <algorithm>
#include <cstdint>

#include <cuda.h>

#include "gnnpre_internal.cuh"

namespace gnnpre {
namespace {

constexpr int kLcTileM = 128;                     // batch rows per tile = accumulator lanes
constexpr int kLcChunk = 32;                      // features per stage: 32 fp32 = one 128-byte swizzle row
constexpr int kLcMaxStages = 8;
constexpr int kLcLookahead = 3;                   // chunks a producer thread keeps in flight beyond the one it announces
constexpr int kLcPipeBytes = 192 * 1024;          // operand stages plus, when it fits, the resident weight
constexpr int kLcResidentMax = 128 * 1024;        // largest weight kept in shared memory for the whole launch
constexpr int kLcEpiBytes = 32 * 128;             // one [32, 32] fp32 output box
constexpr int kLcMaxHidden = 256;                 // N of one MMA, columns of one accumulator buffer
constexpr int kLcABytes = kLcTileM * 128;         // 16 KB
constexpr int kLcProducerWarps = 4;
constexpr int kLcProducerThreads = 32 * kLcProducerWarps;
constexpr int kLcMmaWarp = kLcProducerWarps;       // warps: 0-3 producers, 4 MMA, 5-12 epilogue
constexpr int kLcThreads = 32 * (kLcProducerWarps + 1 + 8);
constexpr int kLcMaxHops = 8;                     // hop matrices per launch
constexpr uint32_t kLcTmemCols = 512;
constexpr uint32_t kLcSuspendNs = 20000;          // a failed poll parks the warp for up to this long
constexpr uint32_t kLcSpinLimit = 50000;          // polls before a wait gives up (about a second)

struct LcMaps {
    CUtensorMap y[kLcMaxHops];    // [batch_size, hidden] outputs, box [32, 32]
    CUtensorMap w;                // [hidden, F] weight, box [hidden, 32]
};

struct LcArgs {
    const float* hop[kLcMaxHops];  // [n, F] hop matrices, leading dimension ldh
    int64_t ldh;
    int64_t n;
    int32_t feat_dim;
    const int32_t* batch;  // row of the hop matrices for each batch position, or nullptr = identity
    int64_t batch_size;
    int32_t num_hops;
    int32_t tiles_m;       // ceil(batch_size / 128)
    int32_t k_chunks;      // ceil(F / 32)
    int32_t hidden;
    uint64_t relu_mask;    // bit k: apply ReLU to hop k's output
    int32_t* error;
    int32_t stages;        // operand stages in flight
    uint32_t stage_stride; // bytes between stages
    int32_t w_resident;    // the weight is loaded once into shared memory at w_off
    uint32_t w_off;        // offsets from the 1024-byte aligned start of dynamic shared memory
    uint32_t epi_off;
    // the split-operand kernel only
    const float* wt;       // [hidden, F] weight, leading dimension ldw
    int64_t ldw;
    int32_t halves;        // column parts: CTAs with blockIdx.x % halves == h compute columns [h n_half, (h + 1) n_half)
    int32_t n_half;
    uint32_t small_off;    // offset of the low parts inside a stage
    // failure-detection self-test: the producers never announce a chunk, so every wait runs out
    int32_t drop_announcements;
    uint32_t spin_limit;   // polls before a wait gives up
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
__device__ __forceinline__ bool lc_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* error,
                                        uint32_t limit = kLcSpinLimit) {
    for (uint32_t i = 0; i < limit; ++i) {
        if (lc_mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    if (error) atomicExch(error, 1);
    return false;
}

// 16 bytes global -> shared without passing through registers; only the first src_bytes (0..16) are
// read, the rest of the 16 bytes is written as zeros.
__device__ __forceinline__ void lc_copy16(uint32_t dst, const float* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
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

// 32 consecutive accumulator columns of this thread's tensor-memory lane.
__device__ __forceinline__ void lc_tmem_load32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

// Tensor store of one [32 rows, 32 columns] box (128-byte swizzle) from shared memory; rows and
// columns beyond the matrix are clipped by the copy engine.
__device__ __forceinline__ void lc_tile_store(const CUtensorMap* tmap, int x0, int y0, uint32_t src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(tmap)),
                 "r"(src), "r"(x0), "r"(y0)
                 : "memory");
}

// Epilogue role (warps 5-12), shared by both kernels: tiles first, first + step, ...; the accumulator holds
// n_cols columns that go to columns col0 .. col0 + n_cols of Y.  Two warps per quarter of the accumulator's
// lanes: the first four epilogue warps take the even 32-column boxes, the last four the odd ones.
__device__ __forceinline__ void lc_epilogue(const LcMaps& maps, const LcArgs& a, uint32_t tiles0, uint32_t tmem_base,
                                            uint32_t acc_full0, uint32_t acc_empty0, volatile int* abort_flag, int first,
                                            int step, int n_cols, int col0) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ew = warp - kLcMmaWarp - 1;  // 0..7
    const int q = warp & 3;                // tensor-memory lanes 32q .. 32q+31 are the ones this warp may read
    const int half = ew >> 2;
    const uint32_t box = tiles0 + a.epi_off + (uint32_t)ew * kLcEpiBytes;
    const int boxes = (n_cols + 31) / 32;
    const int total_tiles = a.num_hops * a.tiles_m;
    int it = 0;
    for (int t = first; t < total_tiles; t += step, ++it) {
        const int hop = t / a.tiles_m, mt = t - hop * a.tiles_m;
        const int buf = it & 1;
        const uint32_t acc_ph = (uint32_t)(it >> 1) & 1u;
        if (!__all_sync(0xffffffffu, lc_wait(acc_full0 + 8u * buf, acc_ph, abort_flag, a.error, a.spin_limit))) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const bool relu = (a.relu_mask >> hop) & 1u;
        const uint32_t taddr = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)buf * kLcMaxHidden;
        // the read of box i + 2 is in flight while box i is written out
        uint32_t v[2][32];
        if (half < boxes) lc_tmem_load32(taddr + 32u * half, v[0]);
#pragma unroll 2
        for (int i = half, u = 0; i < boxes; i += 2, u ^= 1) {
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (i + 2 < boxes) lc_tmem_load32(taddr + 32u * (i + 2), v[u ^ 1]);
            // the previous store must have read the staging box before it is overwritten
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float4 o = make_float4(__uint_as_float(v[u][4 * j]), __uint_as_float(v[u][4 * j + 1]),
                                       __uint_as_float(v[u][4 * j + 2]), __uint_as_float(v[u][4 * j + 3]));
                if (relu) {
                    o.x = fmaxf(o.x, 0.f);
                    o.y = fmaxf(o.y, 0.f);
                    o.z = fmaxf(o.z, 0.f);
                    o.w = fmaxf(o.w, 0.f);
                }
                // row `lane` of the box, 16-byte piece j, in the 128-byte swizzle (no bank conflicts)
                const uint32_t dst = box + 128u * lane + ((uint32_t)(j ^ (lane & 7)) << 4);
                asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(o.x), "f"(o.y), "f"(o.z), "f"(o.w)
                             : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                lc_tile_store(&maps.y[hop], col0 + 32 * i, mt * kLcTileM + 32 * q, box);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) lc_mbar_arrive(acc_empty0 + 8u * buf);
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    __syncwarp();
}

__global__ void __launch_bounds__(kLcThreads, 1) k_lc_first_layer(const __grid_constant__ LcMaps maps, const LcArgs a) {
    extern __shared__ unsigned char lc_smem[];
    __shared__ __align__(8) unsigned long long bars[2 * kLcMaxStages + 6];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tiles0 = (lc_smem_u32(lc_smem) + 1023u) & ~1023u;  // operand tiles need 1024-byte alignment
    const uint32_t bar0 = lc_smem_u32(&bars[0]);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kLcMaxStages + s); };
    auto acc_full_bar = [&](int b) { return bar0 + 8u * (2 * kLcMaxStages + b); };
    auto acc_empty_bar = [&](int b) { return bar0 + 8u * (2 * kLcMaxStages + 2 + b); };
    const uint32_t drain_bar = bar0 + 8u * (2 * kLcMaxStages + 4);
    const uint32_t w_bar = bar0 + 8u * (2 * kLcMaxStages + 5);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kLcMaxStages; ++s) {
            // every producer thread arrives once its copies have landed; a streamed weight chunk adds
            // one arrival that carries the chunk's byte count
            lc_mbar_init(full_bar(s), kLcProducerThreads + (a.w_resident ? 0 : 1));
            lc_mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            lc_mbar_init(acc_full_bar(b), 1);
            lc_mbar_init(acc_empty_bar(b), 8);  // one arrival per epilogue warp
        }
        lc_mbar_init(drain_bar, 1);
        lc_mbar_init(w_bar, 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kLcMmaWarp) {
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
    const uint32_t w_chunk_bytes = (uint32_t)a.hidden * 128u;

    if (warp < kLcProducerWarps) {
        // ---------------------------------------------------------------- producers
        const int pt = threadIdx.x;  // 0..127
        if (a.w_resident && pt == 0) {  // the whole weight, once: it stays in shared memory for every tile
            lc_mbar_arrive_expect_tx(w_bar, (uint32_t)a.k_chunks * w_chunk_bytes);
            for (int kc = 0; kc < a.k_chunks; ++kc)
                lc_tile_load(tiles0 + a.w_off + (uint32_t)kc * w_chunk_bytes, &maps.w, kc * kLcChunk, 0, w_bar);
        }
        // Eight consecutive lanes copy the eight 16-byte pieces of one row's chunk (128 contiguous bytes);
        // a warp instruction covers four rows, a thread eight rows of its warp's 32.
        const int piece = lane & 7;
        const int row0 = 32 * warp + (lane >> 3);            // this thread's rows: row0 + 4 i, i < 8
        int s = 0;           // stage the next chunk goes to
        uint32_t ph = 0;
        int s_done = 0;      // stage whose copies are announced next
        uint32_t issued = 0, announced = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const int hop = t / a.tiles_m, mt = t - hop * a.tiles_m;
            const float* src_row[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int64_t pos = (int64_t)mt * kLcTileM + row0 + 4 * i;
                int64_t r = -1;
                if (pos < a.batch_size) r = a.batch ? (int64_t)__ldg(a.batch + pos) : pos;
                // rows past the batch and indices outside the matrix are read as zeros (no bytes fetched)
                src_row[i] = (r >= 0 && r < a.n) ? a.hop[hop] + r * a.ldh : nullptr;
            }
            for (int kc = 0; kc < a.k_chunks; ++kc) {
                if (!lc_wait(empty_bar(s), ph ^ 1u, abort_flag, a.error, a.spin_limit)) {
                    ok = false;
                    break;
                }
                const int col = kc * kLcChunk + 4 * piece;
                const int left = a.feat_dim - col;                     // valid floats from col on
                const uint32_t bytes = left >= 4 ? 16u : left > 0 ? 4u * left : 0u;
                const uint32_t a_dst = tiles0 + (uint32_t)s * a.stage_stride;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    // row (row0 + 4 i) of the tile, 16-byte piece `piece`, in the 128-byte swizzle
                    const int row = row0 + 4 * i;
                    const uint32_t dst = a_dst + 128u * row + ((uint32_t)(piece ^ (row & 7)) << 4);
                    const bool live = src_row[i] != nullptr && bytes != 0;
                    lc_copy16(dst, live ? src_row[i] + col : a.hop[hop], live ? bytes : 0u);
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
                if (!a.w_resident && pt == 0) {
                    lc_mbar_arrive_expect_tx(full_bar(s), w_chunk_bytes);
                    lc_tile_load(a_dst + kLcABytes, &maps.w, kc * kLcChunk, 0, full_bar(s));
                }
                ++issued;
                if (++s == a.stages) {
                    s = 0;
                    ph ^= 1u;
                }
                if (issued - announced > (uint32_t)kLcLookahead) {
                    // all but the newest kLcLookahead groups have landed: hand the oldest to the MMA warp
                    asm volatile("cp.async.wait_group %0;" ::"n"(kLcLookahead) : "memory");
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    if (!a.drop_announcements) lc_mbar_arrive(full_bar(s_done));
                    ++announced;
                    if (++s_done == a.stages) s_done = 0;
                }
            }
        }
        // the tail: everything still in flight lands, then the remaining chunks are announced
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        while (announced < issued) {
            if (!a.drop_announcements) lc_mbar_arrive(full_bar(s_done));
            ++announced;
            if (++s_done == a.stages) s_done = 0;
        }
        // tensor copies of the weight land in this CTA's shared memory: wait for them before leaving
        if (pt == 0) {
            if (a.w_resident) {
                for (uint32_t i = 0; i < kLcSpinLimit; ++i)
                    if (lc_mbar_try_wait(w_bar, 0)) break;
            } else {
                for (int back = 0; back < a.stages && (uint32_t)back < issued; ++back) {
                    if (--s < 0) {  // walk the stages backwards from the last one filled
                        s = a.stages - 1;
                        ph ^= 1u;
                    }
                    for (uint32_t i = 0; i < kLcSpinLimit; ++i)
                        if (lc_mbar_try_wait(full_bar(s), ph)) break;
                }
            }
        }
    } else if (warp == kLcMmaWarp) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = lc_instr_desc(a.hidden);
            int s = 0, it = 0;
            uint32_t ph = 0;
            bool ok = !a.w_resident || lc_wait(w_bar, 0, abort_flag, a.error, a.spin_limit);
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
                const int buf = it & 1;
                const uint32_t acc_ph = (uint32_t)(it >> 1) & 1u;
                if (!lc_wait(acc_empty_bar(buf), acc_ph ^ 1u, abort_flag, a.error, a.spin_limit)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmem_d = tmem_base + (uint32_t)buf * kLcMaxHidden;
                for (int kc = 0; kc < a.k_chunks; ++kc) {
                    if (!lc_wait(full_bar(s), ph, abort_flag, a.error, a.spin_limit)) {
                        ok = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_src = tiles0 + (uint32_t)s * a.stage_stride;
                    const uint32_t b_src = a.w_resident ? tiles0 + a.w_off + (uint32_t)kc * w_chunk_bytes : a_src + kLcABytes;
#pragma unroll
                    for (int j = 0; j < kLcChunk / 8; ++j)
                        lc_mma_tf32(tmem_d, lc_operand_desc(a_src + 32u * j), lc_operand_desc(b_src + 32u * j), idesc,
                                    (kc | j) != 0);
                    lc_mma_commit(empty_bar(s));  // the stage is free once these MMAs have read it
                    if (++s == a.stages) {
                        s = 0;
                        ph ^= 1u;
                    }
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
        lc_epilogue(maps, a, tiles0, tmem_base, acc_full_bar(0), acc_empty_bar(0), abort_flag, blockIdx.x, gridDim.x,
                    a.hidden, 0);
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == kLcMmaWarp) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kLcTmemCols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------
// The same stage with fp32-like accuracy ("3 x tf32"): every fp32 operand is split into a high part
// that tf32 holds exactly (low 13 mantissa bits cleared) and a low part (the exact remainder, which the
// tensor core again reads as tf32), and  x w  ~=  xh wh + xl wh + xh wl  with fp32 accumulation; the dropped terms are
// below 2^-21 |x||w|.  Shared memory has to hold both parts of both operands, so a CTA computes at most
// 128 output columns: with hidden > 128, even and odd CTAs take the two column halves and every batch row is
// gathered once per part (the later reads mostly hit L2).  No tensor copies on the input side: the producer
// threads bring rows of the hop matrix AND rows of the weight in with 16-byte asynchronous copies,
// then read their own pieces back, split them and write the two parts (each thread touches only bytes
// it copied itself, so the copy's wait_group is all the synchronisation the split needs).
__device__ __forceinline__ void lc_split_piece(uint32_t big_addr, uint32_t small_addr) {
    // The tensor core ignores the low 13 mantissa bits of an fp32 operand (checked on the device: 1 + 7 * 2^-13
    // enters a product as 1), so the tile as it was copied already acts as the high part; only the low part
    // is computed and stored.
    uint32_t v[4];
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(big_addr) : "memory");
    uint32_t lo[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t hi = v[j] & 0xffffe000u;
        lo[j] = __float_as_uint(__uint_as_float(v[j]) - __uint_as_float(hi));  // exact; read by the tensor core as tf32
    }
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(small_addr), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]) : "memory");
}

__global__ void __launch_bounds__(kLcThreads, 1) k_lc_first_layer_x3(const __grid_constant__ LcMaps maps, const LcArgs a) {
    extern __shared__ unsigned char lc_smem[];
    __shared__ __align__(8) unsigned long long bars[2 * kLcMaxStages + 6];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tiles0 = (lc_smem_u32(lc_smem) + 1023u) & ~1023u;
    const uint32_t bar0 = lc_smem_u32(&bars[0]);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kLcMaxStages + s); };
    auto acc_full_bar = [&](int b) { return bar0 + 8u * (2 * kLcMaxStages + b); };
    auto acc_empty_bar = [&](int b) { return bar0 + 8u * (2 * kLcMaxStages + 2 + b); };
    const uint32_t drain_bar = bar0 + 8u * (2 * kLcMaxStages + 4);
    const uint32_t w_bar = bar0 + 8u * (2 * kLcMaxStages + 5);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kLcMaxStages; ++s) {
            lc_mbar_init(full_bar(s), kLcProducerThreads);
            lc_mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            lc_mbar_init(acc_full_bar(b), 1);
            lc_mbar_init(acc_empty_bar(b), 8);
        }
        lc_mbar_init(drain_bar, 1);
        lc_mbar_init(w_bar, kLcProducerThreads);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kLcMmaWarp) {
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
    const int half = blockIdx.x % a.halves;
    const int first = blockIdx.x / a.halves, step = gridDim.x / a.halves;
    constexpr uint32_t kPart = kLcABytes;               // bytes of one part of the rows' chunk: [128, 32] floats
    const uint32_t w_part = (uint32_t)a.n_half * 128u;  // bytes of one part of the weight's chunk: [n_half, 32] floats

    if (warp < kLcProducerWarps) {
        // ---------------------------------------------------------------- producers
        const int piece = lane & 7;
        const int row0 = 32 * warp + (lane >> 3);  // this thread's rows (of the tile and of the weight half): row0 + 4 i
        const float* w_row[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = row0 + 4 * i;
            w_row[i] = r < a.n_half ? a.wt + (int64_t)(half * a.n_half + r) * a.ldw : nullptr;
        }
        // copy this thread's pieces of chunk kc of `rows` (hop rows or weight rows) to `dst_part`
        // (a part holds row_limit rows: 128 for the tile, n_half for the weight; rows beyond it do not exist)
        auto copy_chunk = [&](const auto& rows, int kc, uint32_t dst_part, int row_limit) {
            const int col = kc * kLcChunk + 4 * piece;
            const int left = a.feat_dim - col;
            const uint32_t bytes = left >= 4 ? 16u : left > 0 ? 4u * left : 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int row = row0 + 4 * i;
                if (row >= row_limit) continue;
                const uint32_t dst = dst_part + 128u * row + ((uint32_t)(piece ^ (row & 7)) << 4);
                const bool live = rows[i] != nullptr && bytes != 0;
                lc_copy16(dst, live ? rows[i] + col : a.wt, live ? bytes : 0u);
            }
        };
        auto split_part = [&](uint32_t big_part, uint32_t small_part, int row_limit) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int row = row0 + 4 * i;
                if (row >= row_limit) continue;
                const uint32_t off = 128u * row + ((uint32_t)(piece ^ (row & 7)) << 4);
                lc_split_piece(big_part + off, small_part + off);
            }
        };
        if (a.w_resident) {  // the weight half, once: both parts stay in shared memory for every tile
            for (int kc = 0; kc < a.k_chunks; ++kc) copy_chunk(w_row, kc, tiles0 + a.w_off + (uint32_t)kc * 2u * w_part, a.n_half);
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            for (int kc = 0; kc < a.k_chunks; ++kc) {
                const uint32_t wb = tiles0 + a.w_off + (uint32_t)kc * 2u * w_part;
                split_part(wb, wb + w_part, a.n_half);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            lc_mbar_arrive(w_bar);
        }
        const uint32_t lookahead = (uint32_t)a.stages - 1u;  // 1, 2 or 3
        int s = 0, s_done = 0;
        uint32_t ph = 0, issued = 0, announced = 0;
        auto announce = [&]() {  // the oldest unannounced chunk has landed: split it and hand it to the MMA warp
            const uint32_t base = tiles0 + (uint32_t)s_done * a.stage_stride;
            split_part(base, base + a.small_off, kLcTileM);
            if (!a.w_resident) split_part(base + kPart, base + a.small_off + kPart, a.n_half);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            lc_mbar_arrive(full_bar(s_done));
            ++announced;
            if (++s_done == a.stages) s_done = 0;
        };
        bool ok = true;
        for (int t = first; t < total_tiles && ok; t += step) {
            const int hop = t / a.tiles_m, mt = t - hop * a.tiles_m;
            const float* src_row[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int64_t pos = (int64_t)mt * kLcTileM + row0 + 4 * i;
                int64_t r = -1;
                if (pos < a.batch_size) r = a.batch ? (int64_t)__ldg(a.batch + pos) : pos;
                src_row[i] = (r >= 0 && r < a.n) ? a.hop[hop] + r * a.ldh : nullptr;
            }
            for (int kc = 0; kc < a.k_chunks; ++kc) {
                if (!lc_wait(empty_bar(s), ph ^ 1u, abort_flag, a.error, a.spin_limit)) {
                    ok = false;
                    break;
                }
                const uint32_t base = tiles0 + (uint32_t)s * a.stage_stride;
                copy_chunk(src_row, kc, base, kLcTileM);
                if (!a.w_resident) copy_chunk(w_row, kc, base + kPart, a.n_half);
                asm volatile("cp.async.commit_group;" ::: "memory");
                ++issued;
                if (++s == a.stages) {
                    s = 0;
                    ph ^= 1u;
                }
                if (issued - announced > lookahead) {
                    if (lookahead == 1u) {
                        asm volatile("cp.async.wait_group 1;" ::: "memory");
                    } else if (lookahead == 2u) {
                        asm volatile("cp.async.wait_group 2;" ::: "memory");
                    } else {
                        asm volatile("cp.async.wait_group 3;" ::: "memory");
                    }
                    announce();
                }
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        while (announced < issued) announce();
    } else if (warp == kLcMmaWarp) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = lc_instr_desc(a.n_half);
            int s = 0, it = 0;
            uint32_t ph = 0;
            bool ok = !a.w_resident || lc_wait(w_bar, 0, abort_flag, a.error, a.spin_limit);
            for (int t = first; t < total_tiles && ok; t += step, ++it) {
                const int buf = it & 1;
                const uint32_t acc_ph = (uint32_t)(it >> 1) & 1u;
                if (!lc_wait(acc_empty_bar(buf), acc_ph ^ 1u, abort_flag, a.error, a.spin_limit)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmem_d = tmem_base + (uint32_t)buf * kLcMaxHidden;
                for (int kc = 0; kc < a.k_chunks; ++kc) {
                    if (!lc_wait(full_bar(s), ph, abort_flag, a.error, a.spin_limit)) {
                        ok = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t base = tiles0 + (uint32_t)s * a.stage_stride;
                    const uint32_t xh = base, xl = base + a.small_off;
                    const uint32_t wh = a.w_resident ? tiles0 + a.w_off + (uint32_t)kc * 2u * w_part : base + kPart;
                    const uint32_t wl = a.w_resident ? wh + w_part : base + a.small_off + kPart;
#pragma unroll
                    for (int j = 0; j < kLcChunk / 8; ++j) {
                        const uint32_t o = 32u * j;
                        // small terms first, the leading term last
                        lc_mma_tf32(tmem_d, lc_operand_desc(xl + o), lc_operand_desc(wh + o), idesc, (kc | j) != 0);
                        lc_mma_tf32(tmem_d, lc_operand_desc(xh + o), lc_operand_desc(wl + o), idesc, 1u);
                        lc_mma_tf32(tmem_d, lc_operand_desc(xh + o), lc_operand_desc(wh + o), idesc, 1u);
                    }
                    lc_mma_commit(empty_bar(s));
                    if (++s == a.stages) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
                if (ok) lc_mma_commit(acc_full_bar(buf));
            }
            lc_mma_commit(drain_bar);
            for (uint32_t i = 0; i < kLcSpinLimit; ++i)
                if (lc_mbar_try_wait(drain_bar, 0)) break;
        }
        __syncwarp();
    } else {
        lc_epilogue(maps, a, tiles0, tmem_base, acc_full_bar(0), acc_empty_bar(0), abort_flag, first, step, a.n_half,
                    half * a.n_half);
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == kLcMmaWarp) {
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

// selftest_polls > 0: the producers announce nothing and every wait gives up after that many polls.
static int lc_launch(const float* const* hops, int32_t num_hops, int64_t n, int64_t feat_dim, int64_t ldh,
                     const int32_t* batch, int64_t batch_size, const float* Wt, int64_t hidden, int64_t ldw, uint64_t relu_mask,
                     int32_t precision, float* Y, int64_t ldy, int64_t y_hop_stride, int32_t* error_flag, void* stream,
                     uint32_t selftest_polls) {
    if (!hops || num_hops < 1 || num_hops > GNNPRE_MAX_HOPS || !Wt || (!Y && batch_size != 0)) return GNNPRE_ERR_INVALID_ARG;
    if (n < 1 || n > INT32_MAX || feat_dim < 1 || feat_dim > INT32_MAX - kLcChunk || batch_size < 0) return GNNPRE_ERR_INVALID_ARG;
    if (precision != GNNPRE_LC_TF32 && precision != GNNPRE_LC_TF32X3) return GNNPRE_ERR_INVALID_ARG;
    if (hidden < 16 || hidden > kLcMaxHidden || hidden % 16 != 0) return GNNPRE_ERR_INVALID_ARG;
    const bool x3 = precision == GNNPRE_LC_TF32X3;
    // Split operands: both parts of a CTA's weight columns must fit in shared memory, so a CTA computes at most 128
    // output columns; each part is a whole number of 32-column boxes.  (Parts of 64 columns leave room for four
    // operand stages instead of two but were measured slower, 8.4 against 4.5 ms on the 2.4 M-row workload: the
    // per-tile hand-offs, not the stage count, set the pace.)
    const int32_t halves = x3 && hidden > 128 ? 2 : 1;
    if (halves == 2 && hidden % 64 != 0) return GNNPRE_ERR_INVALID_ARG;
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

    // Shared memory: [operand stages][resident weight, when it fits][8 warps x 1 output box], after the
    // 1024-byte alignment slack.
    const int32_t k_chunks = (int32_t)((feat_dim + kLcChunk - 1) / kLcChunk);
    const int32_t n_half = (int32_t)(hidden / halves);
    bool resident;
    uint32_t stage_stride, small_off = 0, w_off;
    int32_t stages;
    int64_t w_bytes;
    if (!x3) {
        w_bytes = (int64_t)k_chunks * hidden * 128;
        resident = w_bytes <= kLcResidentMax;
        stage_stride = resident ? (uint32_t)kLcABytes : (uint32_t)(kLcABytes + hidden * 128);
        stages = (int32_t)std::min<int64_t>(kLcMaxStages, (kLcPipeBytes - (resident ? w_bytes : 0)) / stage_stride);
    } else {
        // per chunk a high and a low part of the tile's rows (16 KB each) and of the weight part (n_half x 128 B each)
        const uint32_t w_part = (uint32_t)n_half * 128u;
        w_bytes = (int64_t)k_chunks * 2 * w_part;
        resident = w_bytes <= kLcResidentMax;
        small_off = resident ? (uint32_t)kLcABytes : (uint32_t)kLcABytes + w_part;
        stage_stride = 2u * small_off;
        stages = (int32_t)std::min<int64_t>(4, (kLcPipeBytes - (resident ? w_bytes : 0)) / stage_stride);
    }
    w_off = (uint32_t)stages * stage_stride;
    const uint32_t epi_off = w_off + (resident ? (uint32_t)w_bytes : 0u);
    const size_t smem = 1024 + (size_t)epi_off + 8 * kLcEpiBytes;
    auto kernel = x3 ? k_lc_first_layer_x3 : k_lc_first_layer;
    GNNPRE_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));

    LcMaps maps;
    GNNPRE_TRY(encode_map_2d(Wt, feat_dim, hidden, ldw, kLcChunk, (int)hidden, &maps.w));
    for (int32_t k0 = 0; k0 < num_hops; k0 += kLcMaxHops) {  // at most kLcMaxHops hop matrices ride in one launch
        const int32_t kn = std::min<int32_t>(kLcMaxHops, num_hops - k0);
        LcArgs a;
        for (int32_t k = 0; k < kLcMaxHops; ++k) {
            const int32_t kk = k0 + std::min(k, kn - 1);
            a.hop[k] = hops[kk];
            GNNPRE_TRY(encode_map_2d(Y + (int64_t)kk * y_hop_stride, hidden, batch_size, ldy, 32, 32, &maps.y[k]));
        }
        a.ldh = ldh;
        a.n = n;
        a.feat_dim = (int32_t)feat_dim;
        a.batch = batch;
        a.batch_size = batch_size;
        a.num_hops = kn;
        a.tiles_m = (int32_t)tiles_m;
        a.k_chunks = k_chunks;
        a.hidden = (int32_t)hidden;
        a.relu_mask = relu_mask >> k0;
        a.error = error_flag;
        a.stages = stages;
        a.stage_stride = stage_stride;
        a.w_resident = resident ? 1 : 0;
        a.w_off = w_off;
        a.epi_off = epi_off;
        a.wt = Wt;
        a.ldw = ldw;
        a.halves = halves;
        a.n_half = n_half;
        a.small_off = small_off;
        a.drop_announcements = selftest_polls > 0 ? 1 : 0;
        a.spin_limit = selftest_polls > 0 ? selftest_polls : kLcSpinLimit;
        const int64_t total = (int64_t)kn * tiles_m;
        const unsigned grid = (unsigned)(std::min<int64_t>(num_sms / halves, total) * halves);
        kernel<<<grid, kLcThreads, smem, st>>>(maps, a);
        GNNPRE_CUDA(cudaGetLastError());
    }
    return GNNPRE_OK;
}

extern "C" int gnnpre_lc_first_layer(const float* const* hops, int32_t num_hops, int64_t n, int64_t feat_dim, int64_t ldh,
                                     const int32_t* batch, int64_t batch_size, const float* Wt, int64_t hidden, int64_t ldw,
                                     uint64_t relu_mask, int32_t precision, float* Y, int64_t ldy, int64_t y_hop_stride,
                                     int32_t* error_flag, void* stream) {
    return lc_launch(hops, num_hops, n, feat_dim, ldh, batch, batch_size, Wt, hidden, ldw, relu_mask, precision, Y, ldy,
                     y_hop_stride, error_flag, stream, 0);
}

// Failure-detection self-test: see include/gnnpre.h.
extern "C" int gnnpre_lc_selftest_wait_timeout(const float* hop, int64_t n, int64_t feat_dim, int64_t ldh, const float* Wt,
                                               int64_t hidden, int64_t ldw, float* Y, int64_t ldy, int32_t* error_flag,
                                               uint32_t polls, void* stream) {
    if (!error_flag || polls == 0 || polls > 100000u) return GNNPRE_ERR_INVALID_ARG;
    const float* hops[1] = {hop};
    const int64_t rows = n < kLcTileM ? n : kLcTileM;  // one tile, one CTA
    GNNPRE_CUDA(cudaMemsetAsync(error_flag, 0, sizeof(int32_t), static_cast<cudaStream_t>(stream)));
    const int rc = lc_launch(hops, 1, n, feat_dim, ldh, nullptr, rows, Wt, hidden, ldw, 0, GNNPRE_LC_TF32, Y, ldy, 0, error_flag,
                             stream, polls);
    if (rc != GNNPRE_OK) return rc;
    GNNPRE_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    int32_t flag = 0;
    GNNPRE_CUDA(cudaMemcpy(&flag, error_flag, sizeof(flag), cudaMemcpyDeviceToHost));
    return flag ? GNNPRE_ERR_TIMEOUT : GNNPRE_OK;
}
