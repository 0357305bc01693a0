// Pass 2: re-read the logits once and write
//     dlogits[r, v] = g_n m_r (softmax(z[r, .])_v - 1[v == y_r]),
// the derivative of the Eq. 3 surrogate loss through the log-softmax.
//
// One kernel, HBM-bound.  Persistent CTAs draw rows from a counter, scattered over the block of rows
// (draw t stands for row (t * stride) mod rows, stride coprime to the row count), because the two kinds
// of rows are spread unevenly: masked rows cluster at the end of every generation.
//
//  rows that are masked, or whose coefficient g_n is zero, get zeros and nothing is read: each CTA's
//  producer thread sends them straight from a zeroed shared-memory buffer with bulk shared->global
//  copies -- all of them before it starts on the live rows when the launch is large, between the
//  loads of the live rows when it is small.
//
//  live rows: the producer thread draws rows from the first counter, passes over the dead ones, streams
//  each live row into a ring of shared-memory stages with bulk
//  global->shared copies, running ahead across row boundaries, and publishes the row's number
//  through a small queue.  Eight consumer warps wait on a stage's barrier, turn the logits into
//  dlogits IN PLACE in shared memory, and one of them sends the stage back out with a bulk
//  shared->global copy; the stage returns to the producer once that copy has finished reading it.
//  Bytes in flight are set by the ring, not by registers, and both directions move in bursts of
//  kChunk bytes.  A chunk is fully read before any of it is overwritten, so dlogits may be the
//  logits buffer itself.
//
// The arithmetic of one vector of a row is in dz_rows.cuh (shared with the on-policy kernel).
#include "dz_rows.cuh"
#include "rapid_common.cuh"
#include "tma_pipe.cuh"

#ifndef RAPID_P2_CHUNK
#define RAPID_P2_CHUNK 16384
#endif
#ifndef RAPID_P2_STAGES
#define RAPID_P2_STAGES 6
#endif

namespace rapid {

namespace {

constexpr int kConsumers = 256;
constexpr int kConsumerWarps = kConsumers / 32;
constexpr int kThreads = kConsumers + 32;  // + one producer warp
constexpr int kChunk = RAPID_P2_CHUNK;     // bytes per stage
constexpr int kStages = RAPID_P2_STAGES;
#ifndef RAPID_P2_STOREDEPTH
#define RAPID_P2_STOREDEPTH (RAPID_P2_STAGES / 2)  // measured best: three stages loading, three draining
#endif
constexpr int kStoreDepth = RAPID_P2_STOREDEPTH;  // bulk stores allowed to be reading their stage
static_assert(kStoreDepth >= 1 && kStoreDepth <= kStages - 2, "leave at least two stages for loads");
constexpr int kVecPerChunk = kChunk / 16;
constexpr int kVecPerThread = kVecPerChunk / kConsumers;
static_assert(kVecPerChunk % kConsumers == 0, "chunk must be a multiple of 16 B x consumers");
static_assert(kStages >= 3, "need a stage to load, one to work on and one to store");

constexpr int kZeroBuf = 8192;  // zeroed shared memory that the fills of rows without gradient are sent from

__device__ __forceinline__ bool row_is_live(const Workspace& ws, int64_t r, int seq_len) {
    return ws.row_state[r] == ROW_OK && ws.coef[(int)(r / seq_len)] != 0.0;
}

// ---- the kernel --------------------------------------------------------------------------------------

template <int DT>
__global__ void __launch_bounds__(kThreads)
dlogits_kernel(const void* logits, void* dlogits /* may alias logits */, int64_t ld, int vocab,
               int seq_len, int64_t row0, int64_t n_rows, const int32_t* __restrict__ targets,
               rapid_stats_t* stats_user, unsigned int* ticket /* two counters, zero at launch */,
               unsigned long long stride, int fill_first, Workspace ws) {
    constexpr int ESIZE = (DT == RAPID_BF16) ? 2 : 4;
    constexpr int PER = 16 / ESIZE;  // elements per 16-byte vector
    using RowConst = typename std::conditional<DT == RAPID_BF16, RowConstBf16, RowConstF32>::type;

    extern __shared__ __align__(128) uint8_t ring[];  // kStages x kChunk, then kZeroBuf zeros
    uint8_t* zeros = ring + (size_t)kStages * kChunk;
    __shared__ __align__(8) uint64_t full_bar[kStages];
    __shared__ __align__(8) uint64_t empty_bar[kStages];
    __shared__ int abort_flag;
    // rows the producer has drawn, in the order it loads them; -1 = no more.  The producer is at most
    // kStages chunks, hence kStages rows, ahead of the consumers.
    constexpr int kRowQ = kStages + 1;
    __shared__ long long row_q[kRowQ];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        abort_flag = 0;
        mbar_init_fence();
    }
    for (int i = tid; i < kZeroBuf / 16; i += kThreads) reinterpret_cast<uint4*>(zeros)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
    __syncthreads();
    volatile int* abortp = &abort_flag;

    // bytes of a row that are loaded: the vocabulary rounded up to whole 16-byte vectors (the
    // pitch is a multiple of 16 bytes and >= vocab, so this stays inside the row); bytes that are
    // stored in bulk: the whole vectors of real columns only
    const int load_bytes = ((vocab * ESIZE + 15) / 16) * 16;
    const int n_chunks = (load_bytes + kChunk - 1) / kChunk;
    const int nvec_row = vocab / PER;

    if (warp == kConsumerWarps) {
        // ------------------------------- producer -------------------------------------------
        if (lane == 0) {
            const int whole = nvec_row * 16;  // bytes of a row in whole vectors of real columns
            auto zero_fill = [&](int64_t i) {
                uint8_t* zrow = static_cast<uint8_t*>(dlogits) + (size_t)i * ld * ESIZE;
                for (int o = 0; o < whole; o += kZeroBuf) bulk_store(zrow + o, zeros, (uint32_t)min(kZeroBuf, whole - o));
                bulk_commit();
                for (int e = nvec_row * PER; e < vocab; ++e) {  // fewer than one vector of columns after them
                    if (ESIZE == 2) reinterpret_cast<uint16_t*>(zrow)[e] = 0;
                    else reinterpret_cast<float*>(zrow)[e] = 0.f;
                }
                bulk_wait_read<4>();  // a few rows' worth of copies in flight is plenty
            };
            // fill_first: the rows without gradient come first, drawn from the second counter, as a pure
            // write stream; no grid-wide barrier separates the two phases, a CTA goes on to the live rows
            // as soon as the dead ones have run out.  Otherwise they are filled as they are drawn, between
            // the loads of the live rows.  (See the launcher for when which.)
            if (fill_first) {
                for (;;) {
                    const unsigned int t = atomicAdd(ticket + 1, 1u);
                    if ((int64_t)t >= n_rows) break;
                    if (!row_is_live(ws, row0 + (int64_t)t, seq_len)) zero_fill((int64_t)t);
                }
            }
            uint32_t it = 0, j = 0;
            bool ok = true;
            auto stage_free = [&](uint32_t k) {  // the stage that load k goes into has been given back
                const uint32_t use = k / kStages;
                return use == 0 || mbar_wait_bounded(&empty_bar[k % kStages], (use & 1u) ^ 1u, abortp);
            };
            while (ok) {
                const unsigned int t = atomicAdd(ticket, 1u);
                if ((int64_t)t >= n_rows) break;
                const int64_t i = (int64_t)(((unsigned long long)t * stride) % (unsigned long long)n_rows);
                if (!row_is_live(ws, row0 + i, seq_len)) {
                    if (!fill_first) zero_fill(i);
                    continue;
                }
                const uint8_t* src = static_cast<const uint8_t*>(logits) + (size_t)i * ld * ESIZE;
                for (int c = 0; c < n_chunks; ++c, ++it) {
                    const int s = it % kStages;
                    if (!stage_free(it)) {
                        ok = false;
                        break;
                    }
                    if (c == 0) row_q[j++ % kRowQ] = i;  // published by the arrive below (release)
                    const int bytes = min(kChunk, load_bytes - c * kChunk);
                    mbar_arrive_expect_tx(&full_bar[s], (uint32_t)bytes);
                    bulk_load(ring + (size_t)s * kChunk, src + (size_t)c * kChunk, (uint32_t)bytes,
                              &full_bar[s]);
                }
            }
            if (ok && stage_free(it)) {  // tell the consumers that this was the last row
                row_q[j % kRowQ] = -1;
                mbar_arrive(&full_bar[it % kStages]);
            }
            if (!ok || *abortp) {
                // gave up: let the copies already issued land before the CTA's memory goes away
                const uint32_t first = it > (uint32_t)kStages ? it - kStages : 0u;
                for (uint32_t k = first; k < it; ++k) {
                    const unsigned long long t0 = global_timer_ns();
                    while (!mbar_try_wait(&full_bar[k % kStages], (k / kStages) & 1u))
                        if (global_timer_ns() - t0 > kWaitLimitNs) break;
                }
            }
            bulk_wait_all<0>();  // the zero buffer must outlive every copy that reads it
        }
    } else {
        // ------------------------------- consumers ------------------------------------------
        uint32_t it = 0;
        bool ok = true;
        for (uint32_t j = 0; ok; ++j) {
            // the row's first chunk (or the end mark) is what tells which row this is; whether it came is
            // settled by all consumers together, so that the decision to go on, stop or give up is uniform
            bool got = mbar_wait_bounded(&full_bar[it % kStages], (it / kStages) & 1u, abortp);
            if (consumer_barrier_or<kConsumers>(!got || *abortp != 0)) break;
            const int64_t i = (int64_t)row_q[j % kRowQ];
            if (i < 0) break;
            const int64_t r = row0 + i;
            const int n = (int)(r / seq_len);
            const double g = ws.coef[n];
            uint8_t* orow = static_cast<uint8_t*>(dlogits) + (size_t)i * ld * ESIZE;
            RowConst rc;
            if constexpr (DT == RAPID_BF16) {
                rc.c = (float)fma(-ws.lse[r], kLog2eD, ws.coef_log2[n]);
                rc.g = (float)g;
                rc.sign2 = (g < 0.0) ? 0x80008000u : 0u;
                rc.y = targets[r];
            } else {
                rc.M = ws.row_max[r];
                rc.a = (float)(ws.lse[r] - (double)rc.M);
                rc.g = (float)g;
                rc.y = targets[r];
            }
            for (int c = 0; c < n_chunks; ++c, ++it) {
                const int s = it % kStages;
                // A wait that gives up raises the abort flag; the thread still goes to the barrier
                // below, which ORs every consumer's view, so all leave together.
                if (c > 0) got = mbar_wait_bounded(&full_bar[s], (it / kStages) & 1u, abortp);
                uint4* sv = reinterpret_cast<uint4*>(ring + (size_t)s * kChunk);
                const int v0 = c * kVecPerChunk;                  // first vector of the chunk in the row
                const int nv = min(kVecPerChunk, nvec_row - v0);  // whole real vectors in the chunk
                if (got) {
                    // ragged tail of the row (fewer than one vector of real columns), before the
                    // stage is overwritten
                    if (c == n_chunks - 1) {
                        const int e = nvec_row * PER + tid;
                        if (e < vocab) dz_scalar(sv, orow, e - v0 * PER, e, rc);
                    }
                    uint4 z[kVecPerThread];
#pragma unroll
                    for (int jj = 0; jj < kVecPerThread; ++jj) {
                        const int v = tid + jj * kConsumers;
                        if (v < nv) z[jj] = sv[v];
                    }
#pragma unroll
                    for (int jj = 0; jj < kVecPerThread; ++jj) {
                        const int v = tid + jj * kConsumers;
                        if (v < nv) sv[v] = dz_vec_any(z[jj], (v0 + v) * PER, rc);
                    }
                    fence_proxy_async_smem();  // generic writes above -> asynchronous read below
                }
                if (consumer_barrier_or<kConsumers>(!got || *abortp != 0)) {
                    ok = false;
                    break;
                }
                if (tid == 0) {
                    if (nv > 0) bulk_store(orow + (size_t)c * kChunk, sv, (uint32_t)nv * 16u);
                    bulk_commit();
                    // the store committed kStoreDepth chunks ago has finished reading its stage
                    bulk_wait_read<kStoreDepth>();
                    if (it >= (uint32_t)kStoreDepth) mbar_arrive(&empty_bar[(it - kStoreDepth) % kStages]);
                }
            }
        }
        if (tid == 0) bulk_wait_all<0>();
    }
    __syncthreads();
    if (tid == 0 && abort_flag) {
        atomicMax(&ws.stats->status, (int)RAPID_ERR_TIMEOUT);
        if (stats_user) atomicMax(&stats_user->status, (int)RAPID_ERR_TIMEOUT);
    }
}

template <int DT>
cudaError_t launch_one(const rapid_desc_t& d, const void* logits_chunk, void* dlogits_chunk,
                       int64_t row0, int64_t n_rows, const int32_t* targets, rapid_stats_t* stats_user,
                       const Workspace& ws, int sm_count, cudaStream_t stream) {
    constexpr size_t smem = (size_t)kStages * kChunk + kZeroBuf;
    cudaError_t e = cudaFuncSetAttribute(dlogits_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dlogits_kernel<DT>, kThreads, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    int64_t grid = (int64_t)sm_count * per_sm;
    if (grid > n_rows) grid = n_rows;
    if (n_rows > 0xffffffffll) return cudaErrorInvalidValue;  // the row counter is 32 bits wide
    e = cudaMemsetAsync(ws.row_ticket, 0, 2 * sizeof(unsigned int), stream);
    if (e != cudaSuccess) return e;
    // HBM moves more bytes per second when the write-only zero fills come first and the read+write traffic
    // of the live rows after them than when the two are mixed (64 x 1024 x 151936 bf16 in one launch: 4.83
    // against 4.92 ms).  A short launch has no time for two ramp-ups, and there filling the dead rows
    // between the loads wins (64 x 4096 x 32000 fp32 in 16 launches of 2 GB: 7.75 against 8.07 ms).
    const int fill_first = (double)n_rows * (double)d.vocab * ((DT == RAPID_BF16) ? 2.0 : 4.0) >= 8.0e9 ? 1 : 0;
    dlogits_kernel<DT><<<(unsigned)grid, kThreads, smem, stream>>>(logits_chunk, dlogits_chunk, d.ld, d.vocab, d.seq_len,
                                                                  row0, n_rows, targets, stats_user, ws.row_ticket,
                                                                  scatter_stride(n_rows), fill_first, ws);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_dlogits(const rapid_desc_t& d, const void* logits_chunk, void* dlogits_chunk,
                           int64_t row0, int64_t n_rows, const int32_t* targets,
                           rapid_stats_t* stats_user, const Workspace& ws, int sm_count,
                           cudaStream_t stream) {
    if (n_rows <= 0) return cudaSuccess;
    if (d.dtype == RAPID_BF16)
        return launch_one<RAPID_BF16>(d, logits_chunk, dlogits_chunk, row0, n_rows, targets, stats_user,
                                      ws, sm_count, stream);
    return launch_one<RAPID_F32>(d, logits_chunk, dlogits_chunk, row0, n_rows, targets, stats_user, ws,
                                 sm_count, stream);
}

}  // namespace rapid
