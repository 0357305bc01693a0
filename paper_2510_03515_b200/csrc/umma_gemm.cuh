// A persistent bf16 GEMM main loop on the 5th-generation tensor cores (tcgen05) with the
// accumulator in tensor memory, used by the fused LM-head path: D[m, n] = sum_k A[m, k] B[n, k].
//
//   * one CTA per SM, 192 threads: warp 0 = TMA producer, warp 1 = MMA issuer (one elected
//     thread) and owner of the tensor-memory allocation, warps 2..5 = epilogue (each reads the 32
//     accumulator lanes its position in the warpgroup gives it access to)
//   * tile 128 x 256, K in blocks of 64 bf16 (one 128-byte swizzle atom); operands arrive by tiled
//     TMA loads (128-byte swizzle) in a ring of kStages stages tracked by mbarriers
//   * two 256-column accumulators in tensor memory, so the epilogue of tile i overlaps the MMAs of
//     tile i + 1
//   * either operand may be K-major (K contiguous in global memory) or MN-major
//   * the epilogue is a functor; it reads the accumulator with tcgen05.ld and does whatever the
//     caller needs (row statistics, dlogits, plain stores)
//
// One CTA per tile and one destination per copy (no clusters); nothing crosses to another GPU.  Every wait is bounded: on a timeout
// the CTA raises an abort flag, all roles leave their loops, outstanding copies and MMAs are given
// a bounded time to land, tensor memory is freed and *status is raised to RAPID_ERR_TIMEOUT.
#pragma once

#include <cuda.h>  // CUtensorMap (types only; the encoder is fetched from the driver at run time)
#include <cuda_runtime.h>
#include <stdint.h>

#include "rapid_pg.h"
#include "tma_pipe.cuh"

namespace rapid {
namespace umma {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int kStages = 4;
constexpr int kABytes = BM * BK * 2;
constexpr int kBBytes = BN * BK * 2;
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kThreads = 192;
constexpr int kEpiThreads = 128;
constexpr int kTmemCols = 512;
constexpr int kEpiStageBytes = 8192;  // per epilogue warp: two 4 KB buffers for outgoing TMA stores
constexpr size_t kSmemBytes = (size_t)kStages * kStageBytes + 4 * kEpiStageBytes + 1024;  // + slack to align to 1024

enum TileOrder : int { M_FASTEST = 0, N_FASTEST = 1 };

struct Shape {
    int m_blocks, n_blocks, k_blocks;
    int order;
};

// ---- PTX wrappers ----------------------------------------------------------------------------------

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], "
        "[%2];" ::"r"(smem_u32(smem_dst)),
        "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t* slot_in_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot_in_smem)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]; one thread issues
__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrive on `bar` once every MMA issued so far by this thread has completed
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp gets lane (base lane + t)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// shared -> global tiled store of one box (clipped at the tensor's bounds), tracked by the issuing
// thread's bulk group.  x * element size must be a multiple of 16 bytes and never negative.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, const void* smem_src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map),
                 "r"(smem_u32(smem_src)), "r"(x), "r"(y)
                 : "memory");
}

// the same, adding the box to what global memory holds (element type taken from the tensor map)
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, const void* smem_src, int x, int y) {
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map),
                 "r"(smem_u32(smem_src)), "r"(x), "r"(y)
                 : "memory");
}

// Byte offset, inside a 128-byte-swizzled box whose rows are 128 bytes, of 16-byte chunk `chunk`
// (0..7) of row `row`: the chunk index is XORed with the row index modulo 8.
__device__ __forceinline__ uint32_t swz128(int row, int chunk) {
    return (uint32_t)row * 128u + (uint32_t)((chunk ^ (row & 7)) << 4);
}

// ---- descriptors -----------------------------------------------------------------------------------

// Shared-memory operand descriptor, 128-byte swizzle.  Fields (bit positions): start address >> 4
// (0-13), leading-dimension byte offset >> 4 (16-29), stride-dimension byte offset >> 4 (32-45),
// descriptor version 1 (46-47), swizzle mode 2 = 128 B (61-63).
//   K-major tile  : rows of 128 bytes (64 bf16 along K); groups of 8 rows are 1024 bytes apart
//                   (stride offset); the leading offset is not used by the hardware in this mode.
//   MN-major tile : rows of 128 bytes hold 64 bf16 along M (or N), one row per k; groups of 8 k-rows
//                   are 1024 bytes apart (stride offset); the next 64 elements along M/N start
//                   `lbo_bytes` further on (leading offset).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor of kind::f16: D = f32 (bits 4-5 = 1), A = B = bf16 (bits 7-9, 10-12 = 1),
// operand majors (bit 15: A, bit 16: B; 0 = K-major, 1 = MN-major), N >> 3 (17-22), M >> 4 (24-28).
__host__ __device__ constexpr uint32_t instr_desc(bool a_mn, bool b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

// ---- the kernel ------------------------------------------------------------------------------------

// Epi must provide:
//   struct Params;                                    (trivially copyable; passed __grid_constant__, so
//                                                      a CUtensorMap member may be handed to TMA)
//   __device__ Epi(const Params&, uint8_t* stage, int quarter, int lane);
//   __device__ void tile(int m0, int n0, uint32_t taddr);
//   __device__ void finish();
// One object lives per epilogue warp for the whole kernel.  `stage` is that warp's kEpiStageBytes
// of shared memory (1024-byte aligned).  `taddr` addresses this warp's 32 accumulator lanes
// (rows m0 + 32 * quarter + lane), column 0 of the tile; the functor reads it with
// tmem_ld32(taddr + column, ...) and every load must have been waited for (tmem_ld_wait) before
// tile() returns.  All 32 lanes call tile() and finish() together.
template <class Epi, bool A_MN, bool B_MN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, Shape shape,
            int* status, const __grid_constant__ typename Epi::Params ep) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t full_bar[kStages];
    __shared__ __align__(8) uint64_t empty_bar[kStages];
    __shared__ __align__(8) uint64_t tfull_bar[2];
    __shared__ __align__(8) uint64_t tempty_bar[2];
    __shared__ __align__(8) uint64_t drain_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&tfull_bar[a], 1);
            mbar_init(&tempty_bar[a], 4);  // one arrival per epilogue warp
        }
        mbar_init(&drain_bar, 1);
        abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 1) {
        tmem_alloc(&tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    volatile int* abortp = &abort_flag;

    const int total = shape.m_blocks * shape.n_blocks;
    const int KB = shape.k_blocks;
    auto decode = [&](int idx, int& mb, int& nb) {
        if (shape.order == M_FASTEST) {
            nb = idx / shape.m_blocks;
            mb = idx - nb * shape.m_blocks;
        } else {
            mb = idx / shape.n_blocks;
            nb = idx - mb * shape.n_blocks;
        }
    };

    if (warp == 0) {
        // ------------------------------------ TMA producer -------------------------------------------
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int idx = blockIdx.x; idx < total && ok; idx += gridDim.x) {
                int mb, nb;
                decode(idx, mb, nb);
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t use = it / kStages;
                    if (use > 0 && !mbar_wait_bounded(&empty_bar[s], (use & 1u) ^ 1u, abortp)) {
                        ok = false;
                        break;
                    }
                    uint8_t* sa = smem + (size_t)s * kStageBytes;
                    uint8_t* sb = sa + kABytes;
                    mbar_arrive_expect_tx(&full_bar[s], (uint32_t)kStageBytes);
                    if (A_MN) {
#pragma unroll
                        for (int j = 0; j < BM / 64; ++j)
                            tma_load_2d(sa + j * (BK * 128), &tmA, mb * BM + j * 64, kb * BK, &full_bar[s]);
                    } else {
                        tma_load_2d(sa, &tmA, kb * BK, mb * BM, &full_bar[s]);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int j = 0; j < BN / 64; ++j)
                            tma_load_2d(sb + j * (BK * 128), &tmB, nb * BN + j * 64, kb * BK, &full_bar[s]);
                    } else {
                        tma_load_2d(sb, &tmB, kb * BK, nb * BN, &full_bar[s]);
                    }
                }
            }
            if (!ok || *abortp) {
                // gave up: let the copies already issued land before the CTA's memory goes away
                const uint32_t first = it > (uint32_t)kStages ? it - kStages : 0u;
                for (uint32_t j = first; j < it; ++j) {
                    const unsigned long long t0 = global_timer_ns();
                    while (!mbar_try_wait(&full_bar[j % kStages], (j / kStages) & 1u))
                        if (global_timer_ns() - t0 > kWaitLimitNs) break;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------ MMA issuer ---------------------------------------------
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(A_MN, B_MN);
            constexpr uint32_t a_step = A_MN ? (UMMA_K * 128) : (UMMA_K * 2);  // bytes per K = 16
            constexpr uint32_t b_step = B_MN ? (UMMA_K * 128) : (UMMA_K * 2);
            constexpr uint32_t a_lbo = A_MN ? (BK * 128) : 16;
            constexpr uint32_t b_lbo = B_MN ? (BK * 128) : 16;
            uint32_t it = 0, tile_iter = 0;
            bool ok = true;
            for (int idx = blockIdx.x; idx < total && ok; idx += gridDim.x, ++tile_iter) {
                const uint32_t acc = tile_iter & 1u, au = tile_iter >> 1;
                if (au > 0 && !mbar_wait_bounded(&tempty_bar[acc], (au & 1u) ^ 1u, abortp)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % kStages;
                    if (!mbar_wait_bounded(&full_bar[s], (it / kStages) & 1u, abortp)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(smem + (size_t)s * kStageBytes);
                    const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
                    for (int ks = 0; ks < BK / UMMA_K; ++ks) {
                        mma_f16(d_tmem, smem_desc(a_addr + ks * a_step, a_lbo), smem_desc(b_addr + ks * b_step, b_lbo),
                                idesc, (kb | ks) != 0 ? 1u : 0u);
                    }
                    mma_commit(&empty_bar[s]);  // the stage is free once these MMAs have read it
                }
                if (ok) mma_commit(&tfull_bar[acc]);
            }
            // every MMA issued has finished before tensor memory is given back
            mma_commit(&drain_bar);
            {
                const unsigned long long t0 = global_timer_ns();
                while (!mbar_try_wait(&drain_bar, 0))
                    if (global_timer_ns() - t0 > kWaitLimitNs) {
                        *abortp = 1;
                        break;
                    }
            }
        }
    } else {
        // ------------------------------------ epilogue ------------------------------------------------
        const int quarter = warp & 3;  // the 32 accumulator lanes this warp may read
        Epi epi(ep, smem + (size_t)kStages * kStageBytes + (size_t)(warp - 2) * kEpiStageBytes, quarter, lane);
        uint32_t tile_iter = 0;
        for (int idx = blockIdx.x; idx < total; idx += gridDim.x, ++tile_iter) {
            int mb, nb;
            decode(idx, mb, nb);
            const uint32_t acc = tile_iter & 1u, au = tile_iter >> 1;
            const bool got = mbar_wait_bounded(&tfull_bar[acc], au & 1u, abortp);
            // the decision to leave is taken per warp, after all lanes have seen the same outcome
            if (!__all_sync(0xffffffffu, got)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
            epi.tile(mb * BM, nb * BN, taddr);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tempty_bar[acc]);
        }
        __syncwarp();
        epi.finish();
    }
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (tid == 0 && abort_flag && status) atomicMax(status, (int)RAPID_ERR_TIMEOUT);
}

// ---- host side -------------------------------------------------------------------------------------

// Tensor map of a row-major bf16 matrix [rows, cols] with pitch `ld` elements (ld * 2 bytes and
// the base must be multiples of 16), for boxes of `box_cols` x `box_rows` with 128-byte swizzle;
// out-of-range elements read as zero.  Returns false if the driver's encoder is unavailable or
// rejects the arguments.
bool make_map_bf16(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
                   uint32_t box_cols, uint32_t box_rows);
// The same for a float matrix (ld * 4 bytes a multiple of 16; box_cols * 4 = 128 bytes).
bool make_map_f32(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
                  uint32_t box_cols, uint32_t box_rows);

template <class Epi, bool A_MN, bool B_MN>
cudaError_t launch_gemm(const CUtensorMap& tmA, const CUtensorMap& tmB, const Shape& shape, int sm_count,
                        int* status, const typename Epi::Params& ep, cudaStream_t stream) {
    auto kern = gemm_kernel<Epi, A_MN, B_MN>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    long long total = (long long)shape.m_blocks * shape.n_blocks;
    if (total <= 0) return cudaSuccess;
    int grid = (int)(total < sm_count ? total : sm_count);
    kern<<<grid, kThreads, kSmemBytes, stream>>>(tmA, tmB, shape, status, ep);
    return cudaGetLastError();
}

}  // namespace umma
}  // namespace rapid
