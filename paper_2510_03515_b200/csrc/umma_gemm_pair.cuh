// The same persistent bf16 GEMM as umma_gemm.cuh, run by PAIRS of CTAs on two SMs of one GPU
// (tcgen05 with cta_group::2): D[m, n] = sum_k A[m, k] B[n, k] in tiles of 256 x 256.
//
//   * a thread-block cluster of two CTAs owns one tile at a time.  CTA r of the pair (r = its rank in
//     the cluster) holds rows [128 r, 128 r + 128) of the tile's A operand and columns
//     [128 r, 128 r + 128) of its B operand in its own shared memory, and rows [128 r, 128 r + 128) of
//     the accumulator, all 256 columns, in its own tensor memory.  One thread of CTA 0 issues every
//     MMA; the tensor cores of both SMs read A from their own SM and B from both.  Per 64-wide K block
//     a CTA therefore loads 32 KB instead of the 48 KB a lone CTA needs for a 128 x 256 tile: a third
//     less shared-memory fill per flop, and a six-stage ring in the same shared memory.
//   * every load is an ordinary tiled TMA load with ONE destination, the issuing CTA's own shared
//     memory (no multicast); the load only reports its bytes on CTA 0's "full" barrier, which is what
//     the cta_group::2 form of the copy is for.  Every tensor map covers this GPU's memory only.
//   * CTA 0's MMA thread frees a stage, and publishes an accumulator, in both CTAs at once
//     (tcgen05.commit with a two-CTA mask); the epilogue warps of both CTAs hand an accumulator back by
//     arriving on CTA 0's barrier.
//   * roles, epilogue functors, tile order and the double-buffered accumulator are those of the
//     single-CTA kernel; the functor of CTA r sees m0 = 256 mb + 128 r.
//
// Every wait is bounded.  On a timeout a CTA raises its abort flag and its roles leave their loops; its
// peer runs into its own limits a few seconds later; both meet at the cluster barrier at the end, after
// which tensor memory is freed and *status is raised to RAPID_ERR_TIMEOUT.
#pragma once

#include "umma_gemm.cuh"

namespace rapid {
namespace umma {

constexpr int kPairStages = 6;
constexpr int kPairABytes = BM * BK * 2;                    // this CTA's 128 rows of A
constexpr int kPairBBytes = (BN / 2) * BK * 2;              // this CTA's 128 of the tile's 256 columns of B
constexpr int kPairStageBytes = kPairABytes + kPairBBytes;  // 32 KB
constexpr size_t kPairSmemBytes = (size_t)kPairStages * kPairStageBytes + 4 * kEpiStageBytes + 1024;

// ---- PTX wrappers ----------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// the address, in the cluster's shared-memory window, of `smem_addr` (a shared::cta address) in CTA `rank`
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Tiled load into THIS CTA's shared memory whose bytes are reported on a barrier of the pair's CTA 0
// (`bar_cluster_addr`, from map_to_cta).  One destination; no multicast.
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* map, int x, int y,
                                                 uint32_t bar_cluster_addr) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], "
        "[%2];" ::"r"(smem_u32(smem_dst)),
        "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y)
        : "memory");
}

__device__ __forceinline__ void tmem_alloc_pair(uint32_t* slot_in_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot_in_smem)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// D[tmem of both CTAs] (+)= A * B over the pair; one thread of CTA 0 issues
__device__ __forceinline__ void mma_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrive on the barrier at `bar`'s place in BOTH CTAs once every MMA issued so far has completed
__device__ __forceinline__ void mma_commit_both(uint64_t* bar) {
    const uint16_t mask = 3;
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
            smem_u32(bar)),
        "h"(mask)
        : "memory");
}
// the same on this CTA's barrier alone
__device__ __forceinline__ void mma_commit_pair_local(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// arrive on a barrier of another CTA of the cluster (address from map_to_cta)
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar_cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
// wait (bounded) for a phase whose arrivals come from the other CTA's threads
__device__ __forceinline__ bool mbar_wait_bounded_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    const unsigned long long t0 = global_timer_ns();
    for (uint32_t spin = 0;; ++spin) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(smem_u32(bar)), "r"(parity), "r"(kSuspendHintNs)
            : "memory");
        if (ok) return true;
        if ((spin & 63u) == 63u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                return false;
            }
        }
    }
}

// instruction descriptor of the pair's MMA: as instr_desc(), with M = 256
__host__ __device__ constexpr uint32_t instr_desc_pair(bool a_mn, bool b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
}

// ---- the kernel ------------------------------------------------------------------------------------

// `shape.m_blocks` counts 128-row blocks, as for the single-CTA kernel; a pair takes two at a time.
// tmB's box holds 128 rows of B when B is K-major (half of the single-CTA kernel's box).
template <class Epi, bool A_MN, bool B_MN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, Shape shape,
                 int* status, const __grid_constant__ typename Epi::Params ep) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t full_bar[kPairStages];   // used in CTA 0: both CTAs' loads of a stage have landed
    __shared__ __align__(8) uint64_t empty_bar[kPairStages];  // in each CTA: the MMAs have read the stage
    __shared__ __align__(8) uint64_t tfull_bar[2];            // in each CTA: an accumulator is complete
    __shared__ __align__(8) uint64_t tempty_bar[2];           // used in CTA 0: both CTAs' epilogues are done with it
    __shared__ __align__(8) uint64_t drain_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();
    if (tid == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&tfull_bar[a], 1);
            mbar_init(&tempty_bar[a], 8);  // one arrival per epilogue warp of either CTA
        }
        mbar_init(&drain_bar, 1);
        abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 1) {  // one warp of each CTA, together
        tmem_alloc_pair(&tmem_slot, kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    cluster_sync_all();  // both CTAs' barriers are initialised before either signals the other's
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    volatile int* abortp = &abort_flag;

    const int m_pairs = (shape.m_blocks + 1) / 2;
    const int total = m_pairs * shape.n_blocks;
    const int KB = shape.k_blocks;
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    auto decode = [&](int idx, int& mp, int& nb) {
        if (shape.order == M_FASTEST) {
            nb = idx / m_pairs;
            mp = idx - nb * m_pairs;
        } else {
            mp = idx / shape.n_blocks;
            nb = idx - mp * shape.n_blocks;
        }
    };

    if (warp == 0) {
        // ------------------------------------ TMA producer (each CTA its own halves) ------------------
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int idx = pair; idx < total && ok; idx += n_pairs) {
                int mp, nb;
                decode(idx, mp, nb);
                const int m0 = (mp * 2 + (int)rank) * BM;            // this CTA's rows of A
                const int n0 = nb * BN + (int)rank * (BN / 2);       // this CTA's columns of B
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % kPairStages;
                    const uint32_t use = it / kPairStages;
                    if (use > 0 && !mbar_wait_bounded(&empty_bar[s], (use & 1u) ^ 1u, abortp)) {
                        ok = false;
                        break;
                    }
                    uint8_t* sa = smem + (size_t)s * kPairStageBytes;
                    uint8_t* sb = sa + kPairABytes;
                    const uint32_t lead_full = map_to_cta(smem_u32(&full_bar[s]), 0);
                    if (rank == 0) mbar_arrive_expect_tx(&full_bar[s], 2u * (uint32_t)kPairStageBytes);
                    if (A_MN) {
#pragma unroll
                        for (int j = 0; j < BM / 64; ++j)
                            tma_load_2d_pair(sa + j * (BK * 128), &tmA, m0 + j * 64, kb * BK, lead_full);
                    } else {
                        tma_load_2d_pair(sa, &tmA, kb * BK, m0, lead_full);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int j = 0; j < (BN / 2) / 64; ++j)
                            tma_load_2d_pair(sb + j * (BK * 128), &tmB, n0 + j * 64, kb * BK, lead_full);
                    } else {
                        tma_load_2d_pair(sb, &tmB, kb * BK, n0, lead_full);
                    }
                }
            }
            if (!ok || *abortp) {
                // gave up: let the copies already issued land before the CTA's memory goes away.  CTA 0
                // sees them on its own barriers; CTA 1's copies report there too, so it just waits a
                // while (a copy takes microseconds).
                if (rank == 0) {
                    const uint32_t first = it > (uint32_t)kPairStages ? it - kPairStages : 0u;
                    for (uint32_t j = first; j < it; ++j) {
                        const unsigned long long t0 = global_timer_ns();
                        while (!mbar_try_wait(&full_bar[j % kPairStages], (j / kPairStages) & 1u))
                            if (global_timer_ns() - t0 > kWaitLimitNs) break;
                    }
                } else {
                    const unsigned long long t0 = global_timer_ns();
                    while (global_timer_ns() - t0 < 2000000ull) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------ MMA issuer (CTA 0 only) ---------------------------------
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = instr_desc_pair(A_MN, B_MN);
            constexpr uint32_t a_step = A_MN ? (UMMA_K * 128) : (UMMA_K * 2);  // bytes per K = 16
            constexpr uint32_t b_step = B_MN ? (UMMA_K * 128) : (UMMA_K * 2);
            constexpr uint32_t a_lbo = A_MN ? (BK * 128) : 16;
            constexpr uint32_t b_lbo = B_MN ? (BK * 128) : 16;
            uint32_t it = 0, tile_iter = 0;
            bool ok = true;
            for (int idx = pair; idx < total && ok; idx += n_pairs, ++tile_iter) {
                const uint32_t acc = tile_iter & 1u, au = tile_iter >> 1;
                if (au > 0 && !mbar_wait_bounded_cluster(&tempty_bar[acc], (au & 1u) ^ 1u, abortp)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % kPairStages;
                    if (!mbar_wait_bounded(&full_bar[s], (it / kPairStages) & 1u, abortp)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(smem + (size_t)s * kPairStageBytes);
                    const uint32_t b_addr = a_addr + kPairABytes;
#pragma unroll
                    for (int ks = 0; ks < BK / UMMA_K; ++ks) {
                        mma_f16_pair(d_tmem, smem_desc(a_addr + ks * a_step, a_lbo), smem_desc(b_addr + ks * b_step, b_lbo),
                                     idesc, (kb | ks) != 0 ? 1u : 0u);
                    }
                    mma_commit_both(&empty_bar[s]);  // the stage is free, in both CTAs, once these MMAs have read it
                }
                if (ok) mma_commit_both(&tfull_bar[acc]);
            }
            // every MMA issued has finished before tensor memory is given back
            mma_commit_pair_local(&drain_bar);
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
        // ------------------------------------ epilogue (each CTA its own 128 rows) --------------------
        const int quarter = warp & 3;  // the 32 accumulator lanes this warp may read
        Epi epi(ep, smem + (size_t)kPairStages * kPairStageBytes + (size_t)(warp - 2) * kEpiStageBytes, quarter, lane);
        uint32_t tile_iter = 0;
        for (int idx = pair; idx < total; idx += n_pairs, ++tile_iter) {
            int mp, nb;
            decode(idx, mp, nb);
            const uint32_t acc = tile_iter & 1u, au = tile_iter >> 1;
            const bool got = mbar_wait_bounded(&tfull_bar[acc], au & 1u, abortp);
            // the decision to leave is taken per warp, after all lanes have seen the same outcome
            if (!__all_sync(0xffffffffu, got)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
            epi.tile((mp * 2 + (int)rank) * BM, nb * BN, taddr);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(map_to_cta(smem_u32(&tempty_bar[acc]), 0));
        }
        __syncwarp();
        epi.finish();
    }
    // neither CTA lets go of its shared or tensor memory while the other may still touch it
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
    if (tid == 0 && abort_flag && status) atomicMax(status, (int)RAPID_ERR_TIMEOUT);
}

// Launch on as many CTA pairs as the device can hold at once (at most one CTA per SM).
template <class Epi, bool A_MN, bool B_MN>
cudaError_t launch_gemm_pair(const CUtensorMap& tmA, const CUtensorMap& tmB, const Shape& shape, int sm_count,
                             int* status, const typename Epi::Params& ep, cudaStream_t stream) {
    auto kern = gemm_pair_kernel<Epi, A_MN, B_MN>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmemBytes);
    if (e != cudaSuccess) return e;
    const long long total = (long long)((shape.m_blocks + 1) / 2) * shape.n_blocks;
    if (total <= 0) return cudaSuccess;
    cudaLaunchAttribute attr = {};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(sm_count & ~1), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kPairSmemBytes;
    cfg.stream = stream;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    e = cudaOccupancyMaxActiveClusters(&clusters, kern, &cfg);
    if (e != cudaSuccess) return e;
    if (clusters < 1) return cudaErrorLaunchOutOfResources;
    long long pairs = clusters < total ? clusters : total;
    cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, shape, status, ep);
}

}  // namespace umma
}  // namespace rapid
