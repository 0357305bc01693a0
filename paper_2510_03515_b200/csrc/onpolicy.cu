// The on-policy special case in ONE pass over the logits: mu = pi_theta, so every importance
// weight is 1 and the estimator is the policy gradient of Eq. 1 with the group advantage of Eq. 2
// (group relative policy gradient, Sec. 3.3).  This is the first inner step of IW-GRPG after the
// behaviour policy has been refreshed (Algorithm 1, "mu <- pi_theta"), and every step of the
// plain PG baseline.
//
// The advantage A_n = R_n - mean_group(R) needs rewards only, so the coefficient g_n = A_n / Z is
// known before any logit is read and a row can be finished as soon as its own log-sum-exp is:
// one HBM read and one write per live row instead of two reads and one write.
//
//   onpolicy_prep_kernel    Eq. 2 advantages, coefficients, token count           (one CTA)
//   onpolicy_rows_kernel    per live row: sweep 1 streams the row through a shared-memory ring
//                           (bulk copies) and accumulates max / sum of exponentials; sweep 2 streams
//                           the same row again -- it was read microseconds ago and mostly still is
//                           in L2 (the second read and all stores carry evict-first hints so that
//                           they do not push it out) -- turns it into dlogits in place in shared
//                           memory and sends it out with bulk stores.  Dead rows (masked, invalid
//                           token, zero coefficient) are zero-filled from a shared-memory zero
//                           buffer, by the producer thread when nobody reads the row.
//   onpolicy_loss_kernel    S_n = sum_t log pi(y_t), loss = - sum_n g_n S_n, statistics (one CTA)
//
// Every wait on a barrier is bounded; a wait that gives up raises RAPID_ERR_TIMEOUT in the
// statistics block and never traps.
#include "dz_rows.cuh"
#include "rapid_common.cuh"
#include "tma_pipe.cuh"

namespace rapid {

namespace {

#ifndef RAPID_OP_CONSUMERS
#define RAPID_OP_CONSUMERS 256
#endif
#ifndef RAPID_OP_CHUNK
#define RAPID_OP_CHUNK 16384
#endif
#ifndef RAPID_OP_STAGES
#define RAPID_OP_STAGES 6
#endif
#ifndef RAPID_OP_HINTS
#define RAPID_OP_HINTS 3  // see policy_evict_last() below; 3 measured best by a small margin
#endif
#ifndef RAPID_OP_F32X2
#define RAPID_OP_F32X2 1  // packed two-float arithmetic in the first sweep (bf16)
#endif
#ifndef RAPID_OP_MINBLOCKS
#define RAPID_OP_MINBLOCKS 2
#endif
constexpr int kConsumers = RAPID_OP_CONSUMERS;
constexpr int kConsumerWarps = kConsumers / 32;
constexpr int kThreads = kConsumers + 32;  // + one producer warp
constexpr int kChunk = RAPID_OP_CHUNK;     // bytes per stage
constexpr int kStages = RAPID_OP_STAGES;
#ifndef RAPID_OP_PENDING
#define RAPID_OP_PENDING 3
#endif
constexpr int kMaxPending = RAPID_OP_PENDING;  // bulk stores that may still be reading their stage
#ifndef RAPID_OP_RETAIN
#define RAPID_OP_RETAIN 0
#endif
// The last kRetain chunks of a row's first sweep are not given back to the producer: they stay in their
// stages, and the second sweep starts on them in place instead of loading them again.  Measured slower at
// every depth (0: 5.79 ms, 1: 5.89, 2: 5.91, 3 with two pending stores: 6.13 on the 64 x 1024 x 151936
// mini-batch): a stage that is held is a stage the ring cannot load into, and that costs more than the
// saved loads bring.  Kept as an option, off.
constexpr int kRetain = RAPID_OP_RETAIN;
static_assert(kRetain >= 0 && kRetain + kMaxPending < RAPID_OP_STAGES, "retained stages, stages that pending stores hold and one to load into");
static_assert(kStages >= kMaxPending + 2, "the ring must keep cycling while stores are in flight");
static_assert((kChunk / 16) % kConsumers == 0, "a chunk is a whole number of 16-byte vectors per consumer");
constexpr int kVecPerChunk = kChunk / 16;
constexpr int kVecPerThread = kVecPerChunk / kConsumers;
constexpr int kVecPerWarp = kVecPerThread * 32;  // a warp's contiguous slice of a chunk, in 16-byte vectors
#ifndef RAPID_OP_ZEROBUF
#define RAPID_OP_ZEROBUF 8192
#endif
constexpr int kZeroBuf = RAPID_OP_ZEROBUF;
constexpr int kPrepThreads = 256;

// L2 cache policies for bulk copies
// RAPID_OP_HINTS: 0 = no preference anywhere; 1 = first sweep evict-last, everything else evict-first;
// 2 = first sweep evict-last, the rest no preference; 3 = first sweep no preference, the rest evict-first
__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
#if RAPID_OP_HINTS == 1 || RAPID_OP_HINTS == 2
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
#else
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
#endif
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
#if RAPID_OP_HINTS == 1 || RAPID_OP_HINTS == 3
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
#else
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
#endif
    return p;
}
__device__ __forceinline__ void bulk_load_hint(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar,
                                               uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::
            "r"(smem_u32(smem_dst)),
        "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void bulk_store_hint(void* gdst, const void* smem_src, uint32_t bytes, uint64_t policy) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::"l"(gdst),
                 "r"(smem_u32(smem_src)), "r"(bytes), "l"(policy)
                 : "memory");
}

__device__ __forceinline__ void consumer_barrier() {
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
}
// ---- before the pass: Eq. 2 advantages and coefficients ------------------------------------------------

__global__ void __launch_bounds__(kPrepThreads)
onpolicy_prep_kernel(int n_seq, int seq_len, int vocab, int n_groups, double norm_z, uint32_t flags,
                     const float* __restrict__ rewards, const int32_t* __restrict__ group_offsets,
                     const int32_t* __restrict__ targets, const uint8_t* __restrict__ mask,
                     float* __restrict__ adv_out, Workspace ws) {
    __shared__ int sh_bad, sh_empty;
    __shared__ long long sh_tok[kPrepThreads / 32];
    const int tid = threadIdx.x;
    if (tid == 0) {
        sh_bad = 0;
        sh_empty = 0;
    }
    __syncthreads();
    for (int k = tid; k <= n_groups; k += kPrepThreads) {
        const int o = group_offsets[k];
        bool bad = (k == 0 && o != 0) || (k == n_groups && o != n_seq) || o < 0 || o > n_seq;
        if (k < n_groups) {
            const int o1 = group_offsets[k + 1];
            if (o1 < o) bad = true;
            if (o1 == o) atomicAdd(&sh_empty, 1);
        }
        if (bad) atomicAdd(&sh_bad, 1);
    }
    // tokens that count (only needed as the normaliser with RAPID_FLAG_NORM_TOKENS)
    long long tok = 0;
    if ((flags & RAPID_FLAG_NORM_TOKENS) && !(flags & RAPID_FLAG_NORM_GIVEN)) {
        const int64_t T = (int64_t)n_seq * seq_len;
        for (int64_t r = tid; r < T; r += kPrepThreads) {
            const bool on = mask ? (mask[r] != 0) : true;
            const int32_t y = targets[r];
            tok += (on && y >= 0 && y < vocab) ? 1 : 0;
        }
    }
    tok = warp_sum(tok);
    if ((tid & 31) == 0) sh_tok[tid >> 5] = tok;
    __syncthreads();
    tok = 0;
    for (int w = 0; w < kPrepThreads / 32; ++w) tok += sh_tok[w];

    if (sh_bad != 0) {
        const float nanf_ = __int_as_float(0x7fc00000);
        for (int n = tid; n < n_seq; n += kPrepThreads) {
            ws.coef[n] = 0.0;
            ws.coef_log2[n] = -INFINITY;
            ws.adv[n] = (double)nanf_;
            if (adv_out) adv_out[n] = nanf_;
        }
        if (tid == 0) {
            ws.stats->status = RAPID_ERR_INVALID_ARG;
            ws.stats->n_empty_group = 0;
        }
        return;
    }
    const double Z = (flags & RAPID_FLAG_NORM_GIVEN)    ? norm_z
                     : (flags & RAPID_FLAG_NORM_TOKENS) ? (double)tok
                                                        : (double)n_seq;
    auto publish = [&](int n, double a) {
        const double g = (Z > 0.0) ? a / Z : 0.0;
        ws.adv[n] = a;
        ws.coef[n] = g;
        ws.coef_log2[n] = (g != 0.0) ? log2(fabs(g)) : -INFINITY;
        ws.weight[n] = 1.0;
        ws.clipped_w[n] = 1.0;
        if (adv_out) adv_out[n] = (float)a;
    };
    if (!(flags & RAPID_FLAG_LEAVE_ONE_OUT)) {
        // one thread per group, members in index order: the plain definition of Eq. 2
        for (int k = tid; k < n_groups; k += kPrepThreads) {
            const int lo = group_offsets[k], hi = group_offsets[k + 1];
            const int Nk = hi - lo;
            if (Nk == 0) continue;
            double sum = 0.0;
            for (int n = lo; n < hi; ++n) sum = __dadd_rn(sum, (double)rewards[n]);
            const double base = __ddiv_rn(sum, (double)Nk);
            for (int n = lo; n < hi; ++n) publish(n, __dsub_rn((double)rewards[n], base));
        }
    } else {
        // leave-one-out: one thread per member, its own index-order sum over the others of its group
        for (int n = tid; n < n_seq; n += kPrepThreads) {
            int a0 = 0, a1 = n_groups;  // the last k with group_offsets[k] <= n
            while (a1 - a0 > 1) {
                const int mid = (a0 + a1) >> 1;
                if (group_offsets[mid] <= n) a0 = mid;
                else a1 = mid;
            }
            const int lo = group_offsets[a0], hi = group_offsets[a0 + 1];
            const int Nk = hi - lo;
            const double R = (double)rewards[n];
            double others = 0.0;
            for (int q = lo; q < hi; ++q)
                if (q != n) others = __dadd_rn(others, (double)rewards[q]);
            double a;
            if (flags & RAPID_FLAG_LOO_LITERAL_DIVISOR) a = __dsub_rn(R, __ddiv_rn(others, (double)Nk));
            else if (Nk > 1) a = __dsub_rn(R, __ddiv_rn(others, (double)(Nk - 1)));
            else a = R;
            publish(n, a);
        }
    }
    if (tid == 0) {
        ws.stats->status = RAPID_OK;
        ws.stats->n_empty_group = sh_empty;
    }
}

// ---- the pass ------------------------------------------------------------------------------------------

// running (max, sum of exponentials) of one thread
struct Acc {
    float m, s0, s1;
};

template <bool FULL>
__device__ __forceinline__ void acc_vec(Acc& a, const uint4 (&q)[kVecPerThread], int nvalid, RowConstBf16*) {
    // bf16: chunk maximum with packed max, then one fused multiply-add and one MUFU exponential per element
    uint32_t mx = 0xff80ff80u;  // (-inf, -inf)
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j)
        if (FULL || j < nvalid)
            mx = bf16x2_max(mx, bf16x2_max(bf16x2_max(q[j].x, q[j].y), bf16x2_max(q[j].z, q[j].w)));
    const float bm = fmaxf(bf16_lo(mx), bf16_hi(mx));
    if (bm > a.m) {
        const float f = ex2_approx((a.m - bm) * kLog2e);
        a.s0 *= f;
        a.s1 *= f;
        a.m = bm;
    }
    // nothing but -inf (or the lowest finite value) so far: no (-inf) - (-inf), no overflow of the shift
    const float nm = (a.m < -1.0e38f) ? 0.f : -a.m * kLog2e;
#if RAPID_OP_F32X2
    // a pair at a time: one packed multiply-add and one packed addition per two logits
    const uint64_t k2 = f32x2(kLog2e, kLog2e), nm2 = f32x2(nm, nm);
    uint64_t s2 = f32x2(a.s0, a.s1);
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j) {
        if (FULL || j < nvalid) {
            const uint32_t w[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float xl, xh;
                f32x2_split(f32x2_fma(f32x2(bf16_lo(w[k]), bf16_hi(w[k])), k2, nm2), xl, xh);
                s2 = f32x2_add(s2, f32x2(ex2_approx(xl), ex2_approx(xh)));
            }
        }
    }
    f32x2_split(s2, a.s0, a.s1);
#else
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j) {
        if (FULL || j < nvalid) {
            const uint32_t w[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                a.s0 += ex2_approx(fmaf(bf16_lo(w[k]), kLog2e, nm));
                a.s1 += ex2_approx(fmaf(bf16_hi(w[k]), kLog2e, nm));
            }
        }
    }
#endif
}
template <bool FULL>
__device__ __forceinline__ void acc_vec(Acc& a, const uint4 (&q)[kVecPerThread], int nvalid, RowConstF32*) {
    float bm = -INFINITY;
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j)
        if (FULL || j < nvalid)
            bm = fmaxf(bm, fmaxf(fmaxf(__uint_as_float(q[j].x), __uint_as_float(q[j].y)),
                                 fmaxf(__uint_as_float(q[j].z), __uint_as_float(q[j].w))));
    if (bm > a.m) {
        const float f = expf(a.m - bm);
        a.s0 *= f;
        a.s1 *= f;
        a.m = bm;
    }
    if (a.m == -INFINITY) return;  // nothing but -inf so far: the sums stay 0
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j) {
        if (FULL || j < nvalid) {
            a.s0 += expf(__uint_as_float(q[j].x) - a.m) + expf(__uint_as_float(q[j].y) - a.m);
            a.s1 += expf(__uint_as_float(q[j].z) - a.m) + expf(__uint_as_float(q[j].w) - a.m);
        }
    }
}
__device__ __forceinline__ void acc_scalar(Acc& a, float z, bool base2) {
    if (z == -INFINITY) return;  // contributes nothing
    if (z > a.m) {
        const float f = base2 ? ex2_approx((a.m - z) * kLog2e) : expf(a.m - z);
        a.s0 *= f;
        a.s1 *= f;
        a.m = z;
    }
    a.s0 += base2 ? ex2_approx((z - a.m) * kLog2e) : expf(z - a.m);
}

// Which sweeps a row gets.  Decided from the inputs alone, identically by every thread.
enum : int { ROWS_NONE = 0, ROWS_STATS = 1, ROWS_BOTH = 2 };
__device__ __forceinline__ int row_plan(int64_t r, int seq_len, int vocab, const int32_t* targets,
                                        const uint8_t* mask, const Workspace& ws, bool want_logp, uint8_t* state) {
    const bool on = mask ? (mask[r] != 0) : true;
    const int32_t y = targets[r];
    if (!on) {
        *state = ROW_MASKED;
        return ROWS_NONE;
    }
    if (y < 0 || y >= vocab) {
        *state = ROW_BAD_TOKEN;
        return ROWS_NONE;
    }
    *state = ROW_OK;
    if (ws.coef[(int)(r / seq_len)] != 0.0) return ROWS_BOTH;
    return want_logp ? ROWS_STATS : ROWS_NONE;
}

template <int DT>
__global__ void __launch_bounds__(kThreads, RAPID_OP_MINBLOCKS)
onpolicy_rows_kernel(const void* logits, void* dlogits /* may alias logits */, int64_t ld, int vocab, int seq_len,
                     int64_t n_rows, const int32_t* __restrict__ targets, const uint8_t* __restrict__ mask,
                     int want_logp, unsigned int* ticket /* two counters, zero at launch */, unsigned long long stride,
                     int fill_first, Workspace ws) {
    constexpr int ESIZE = (DT == RAPID_BF16) ? 2 : 4;
    constexpr int PER = 16 / ESIZE;
    constexpr bool kBase2 = (DT == RAPID_BF16);
    using RowConst = typename std::conditional<DT == RAPID_BF16, RowConstBf16, RowConstF32>::type;

    extern __shared__ __align__(128) uint8_t dyn[];  // kStages x kChunk ring, then kZeroBuf zeros
    uint8_t* ring = dyn;
    uint8_t* zeros = dyn + (size_t)kStages * kChunk;
    __shared__ __align__(8) uint64_t full_bar[kStages];
    __shared__ __align__(8) uint64_t empty_bar[kStages];
    __shared__ int abort_flag;
    __shared__ float sh_m[kConsumerWarps];
    __shared__ double sh_s[kConsumerWarps];
    __shared__ double sh_lse;
    __shared__ float sh_M;
    __shared__ float sh_zy;
    // rows that are read, in the order the producer loads them: 4 * row + plan; -1 = no more.  The
    // producer is at most kStages chunks, hence kStages rows, ahead of the consumers.
    constexpr int kRowQ = kStages + 1;
    __shared__ long long row_q[kRowQ];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kConsumerWarps);  // every consumer warp gives the stage back
        }
        abort_flag = 0;
        mbar_init_fence();
    }
    for (int i = tid; i < kZeroBuf / 16; i += kThreads) reinterpret_cast<uint4*>(zeros)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
    __syncthreads();
    volatile int* abortp = &abort_flag;

    const int load_bytes = ((vocab * ESIZE + 15) / 16) * 16;  // stays inside the row: the pitch is a multiple of 16
    const int n_chunks = (load_bytes + kChunk - 1) / kChunk;
    const int nvec_row = vocab / PER;
    const int whole = nvec_row * 16;  // bytes of a row in whole vectors of real columns
    // Rows are drawn from a counter, so every CTA stays busy until the rows run out however unevenly the
    // rows that are read and the rows that are only zero-filled are spread.  Draw t stands for row
    // (t * stride) mod n_rows, with stride coprime to n_rows and about 0.62 n_rows: rows drawn at about the
    // same time lie far apart, so the memory system sees the batch's average mix of the two kinds rather
    // than one kind after the other (masked rows cluster at the end of every generation).
    auto row_of_draw = [&](unsigned int t) -> int64_t { return (int64_t)(((unsigned long long)t * stride) % (unsigned long long)n_rows); };

    if (warp == kConsumerWarps) {
        // ------------------------------- producer -------------------------------------------
        if (lane == 0) {
            const uint64_t keep = policy_evict_last(), stream = policy_evict_first();
            uint32_t it = 0;
            bool ok = true;
            uint32_t jq = 0;
            auto stage_free = [&](uint32_t k) {  // the stage that load k goes into has been given back
                const uint32_t use = k / kStages;
                return use == 0 || mbar_wait_bounded(&empty_bar[k % kStages], (use & 1u) ^ 1u, abortp);
            };
            // a row nobody reads is finished by this thread alone: zeros from the zero buffer (whole vectors
            // by bulk copies, outside the consumers' accounting of pending stores; the few columns after
            // them one by one) and its entries of the per-row statistics
            auto finish_unread_row = [&](int64_t r, uint8_t st) {
                uint8_t* orow = static_cast<uint8_t*>(dlogits) + (size_t)r * ld * ESIZE;
                for (int o = 0; o < whole; o += kZeroBuf)
                    bulk_store_hint(orow + o, zeros, (uint32_t)min(kZeroBuf, whole - o), stream);
                bulk_commit();
                for (int e = nvec_row * PER; e < vocab; ++e) {
                    if (ESIZE == 2) reinterpret_cast<uint16_t*>(orow)[e] = 0;
                    else reinterpret_cast<float*>(orow)[e] = 0.f;
                }
                ws.row_state[r] = st;
                ws.lse[r] = 0.0;
                ws.token_logp[r] = 0.0;
                ws.row_max[r] = 0.f;
                bulk_wait_read<4>();  // a few rows' worth of copies in flight is plenty
            };
            // fill_first: those rows come first, drawn from the second counter, as a pure write stream;
            // otherwise they are filled as they are drawn, between the loads
            if (fill_first) {
                for (;;) {
                    const unsigned int t = atomicAdd(ticket + 1, 1u);
                    if ((int64_t)t >= n_rows) break;
                    uint8_t st;
                    if (row_plan((int64_t)t, seq_len, vocab, targets, mask, ws, want_logp != 0, &st) == ROWS_NONE)
                        finish_unread_row((int64_t)t, st);
                }
            }
            while (ok) {
                const unsigned int t = atomicAdd(ticket, 1u);
                if ((int64_t)t >= n_rows) break;
                const int64_t r = row_of_draw(t);
                uint8_t st;
                const int plan = row_plan(r, seq_len, vocab, targets, mask, ws, want_logp != 0, &st);
                if (plan == ROWS_NONE) {
                    if (!fill_first) finish_unread_row(r, st);
                    continue;
                }
                const uint8_t* src = static_cast<const uint8_t*>(logits) + (size_t)r * ld * ESIZE;
                for (int sweep = 0; sweep < plan && ok; ++sweep) {
                    // first sweep of a row that will be read again: ask L2 to keep it
                    const uint64_t pol = (sweep == 0 && plan == ROWS_BOTH) ? keep : stream;
                    // the second sweep finds the row's last chunks still in shared memory
                    const int n_load = (sweep == 1) ? n_chunks - min(kRetain, n_chunks) : n_chunks;
                    for (int c = 0; c < n_load; ++c, ++it) {
                        const int s = it % kStages;
                        if (!stage_free(it)) {
                            ok = false;
                            break;
                        }
                        if (sweep == 0 && c == 0) row_q[jq++ % kRowQ] = 4 * r + plan;  // published by the arrive below
                        const int bytes = min(kChunk, load_bytes - c * kChunk);
                        mbar_arrive_expect_tx(&full_bar[s], (uint32_t)bytes);
                        bulk_load_hint(ring + (size_t)s * kChunk, src + (size_t)c * kChunk, (uint32_t)bytes,
                                       &full_bar[s], pol);
                    }
                }
            }
            if (ok && stage_free(it)) {  // tell the consumers that this was the last row
                row_q[jq % kRowQ] = -1;
                mbar_arrive(&full_bar[it % kStages]);
            }
            if (!ok || *abortp) {
                const uint32_t first = it > (uint32_t)kStages ? it - kStages : 0u;
                for (uint32_t j = first; j < it; ++j) {
                    const unsigned long long t0 = global_timer_ns();
                    while (!mbar_try_wait(&full_bar[j % kStages], (j / kStages) & 1u))
                        if (global_timer_ns() - t0 > kWaitLimitNs) break;
                }
            }
            bulk_wait_all<0>();  // the zero fills have left the zero buffer
        }
    } else {
        // ------------------------------- consumers ------------------------------------------
        const uint64_t stream = policy_evict_first();
        int st = 0;         // stage of the next chunk
        uint32_t ph = 0;    // and the phase of its barriers
        bool ok = true;
        auto next_stage = [&]() {
            if (++st == kStages) {
                st = 0;
                ph ^= 1u;
            }
        };
        // stages whose outgoing store may still be reading them, newest first (-1: nothing to release);
        // lane 0 of every warp keeps its own (bulk groups belong to the thread that commits them)
        int pend[kMaxPending];
#pragma unroll
        for (int k = 0; k < kMaxPending; ++k) pend[k] = -2;  // -2: no group at all
        auto release = [&](int s) {
            if (s >= 0) mbar_arrive(&empty_bar[s]);
        };
        // a new bulk group was committed for stage s (or -1 for a zero fill): the group committed
        // kMaxPending groups earlier has finished reading by the time the wait returns
        auto pushed = [&](int s) {
            bulk_wait_read<kMaxPending>();
            release(pend[kMaxPending - 1]);
#pragma unroll
            for (int k = kMaxPending - 1; k > 0; --k) pend[k] = pend[k - 1];
            pend[0] = s;
        };
        // give back the oldest outstanding stage, waiting only for that one store
        auto drain_one = [&]() {
            bool done = false;
#pragma unroll
            for (int i = kMaxPending - 1; i >= 0; --i) {
                if (!done && pend[i] != -2) {
                    switch (i) {
                        case 0: bulk_wait_read<0>(); break;
                        case 1: bulk_wait_read<1>(); break;
                        case 2: bulk_wait_read<2>(); break;
                        case 3: bulk_wait_read<3>(); break;
                        case 4: bulk_wait_read<4>(); break;
                        default: bulk_wait_read<5>(); break;
                    }
                    release(pend[i]);
                    pend[i] = -2;
                    done = true;
                }
            }
        };
        static_assert(kMaxPending >= 1 && kMaxPending <= 6, "drain_one covers up to six pending stores");

        // A row starts when its first chunk has landed; the queue entry published with it says which row
        // it is.  Whether it came is settled by all consumers together: after a timeout a warp stops
        // working (ok = false) but still comes here, where all agree to leave.
        for (uint32_t jq = 0;; ++jq) {
            const bool came = ok && mbar_wait_bounded(&full_bar[st], ph, abortp);
            if (consumer_barrier_or<kConsumers>(!came || *abortp != 0)) break;
            const long long entry = row_q[jq % kRowQ];
            if (entry < 0) break;
            const int64_t r = entry >> 2;
            const int plan = (int)(entry & 3);
            uint8_t* orow = static_cast<uint8_t*>(dlogits) + (size_t)r * ld * ESIZE;
            // rows without gradient get zeros, straight from the zero buffer (after the row has been
            // read, if it is read at all: dlogits may be the logits buffer itself)
            auto zero_row = [&]() {
                if (tid == 0) {
                    for (int o = 0; o < whole; o += kZeroBuf)
                        bulk_store_hint(orow + o, zeros, (uint32_t)min(kZeroBuf, whole - o), stream);
                    bulk_commit();
                    pushed(-1);
                } else if (nvec_row * PER + (tid - 1) < vocab) {
                    if (ESIZE == 2) reinterpret_cast<uint16_t*>(orow)[nvec_row * PER + tid - 1] = 0;
                    else reinterpret_cast<float*>(orow)[nvec_row * PER + tid - 1] = 0.f;
                }
            };
            const int y = targets[r];
            // ---- sweep 1: max and sum of exponentials.  Each warp owns a contiguous slice of every
            // chunk and gives the stage back on its own (the stage's barrier counts the warps), so no
            // CTA-wide barrier is needed per chunk ----
            Acc acc{-INFINITY, 0.f, 0.f};
            const int n_ret = (plan == ROWS_BOTH) ? min(kRetain, n_chunks) : 0;  // chunks kept for the second sweep
            int ret_st = 0;                                                     // stage of the first of them
            if (ok) {
                for (int c = 0; c < n_chunks; ++c) {
                    const int s = st;
                    if (c == n_chunks - n_ret) ret_st = s;
                    const bool got = mbar_wait_bounded(&full_bar[s], ph, abortp);
                    if (__any_sync(0xffffffffu, !got)) {
                        ok = false;
                        break;
                    }
                    next_stage();
                    const uint4* sv = reinterpret_cast<const uint4*>(ring + (size_t)s * kChunk);
                    const int v0 = c * kVecPerChunk;
                    const int nv = min(kVecPerChunk, nvec_row - v0);
                    const uint4* wv = sv + warp * kVecPerWarp + lane;  // this thread's vectors: wv[32 j]
                    const int nvw = nv - warp * kVecPerWarp;           // whole vectors in this warp's slice
                    const bool full = nvw >= kVecPerWarp;              // the same for the whole warp
                    uint4 q[kVecPerThread];
                    int nvalid = 0;
                    if (full) {
#pragma unroll
                        for (int j = 0; j < kVecPerThread; ++j) q[j] = wv[j * 32];
                    } else {
#pragma unroll
                        for (int j = 0; j < kVecPerThread; ++j) {
                            if (j * 32 + lane < nvw) {
                                q[j] = wv[j * 32];
                                nvalid = j + 1;
                            }
                        }
                    }
                    float ztail = 0.f;
                    bool has_tail = false;
                    if (c == n_chunks - 1) {  // ragged tail: fewer than one vector of real columns
                        const int e = nvec_row * PER + tid;
                        if (e < vocab) {
                            const int ei = e - v0 * PER;
                            ztail = (ESIZE == 2)
                                        ? __uint_as_float(((uint32_t) reinterpret_cast<const uint16_t*>(sv)[ei]) << 16)
                                        : reinterpret_cast<const float*>(sv)[ei];
                            has_tail = true;
                        }
                    }
                    const int yi = y - v0 * PER;  // the sampled token's logit
                    if (tid == 0 && yi >= 0 && yi < kVecPerChunk * PER)
                        sh_zy = (ESIZE == 2) ? __uint_as_float(((uint32_t) reinterpret_cast<const uint16_t*>(sv)[yi]) << 16)
                                             : reinterpret_cast<const float*>(sv)[yi];
                    __syncwarp();  // the whole warp has its data in registers: the stage can go (unless it is kept)
                    if (lane == 0) {
                        if (c < n_chunks - n_ret) mbar_arrive(&empty_bar[s]);
                        if (c < kMaxPending) drain_one();  // stages still held by this warp's stores of the previous row
                    }
                    if (full) acc_vec<true>(acc, q, kVecPerThread, (RowConst*)nullptr);
                    else if (nvalid > 0) acc_vec<false>(acc, q, nvalid, (RowConst*)nullptr);
                    if (has_tail) acc_scalar(acc, ztail, kBase2);
                }
            }
            // ---- the row's log-sum-exp, in double; also where all warps agree to leave after a timeout ----
            {
                float m = acc.m, sm = acc.s0 + acc.s1;
                const float wm = warp_max(m);
                sm *= (m == wm) ? 1.f : (kBase2 ? ex2_approx((m - wm) * kLog2e) : expf(m - wm));
                sm = warp_sum(sm);
                if (lane == 0) {
                    sh_m[warp] = wm;
                    sh_s[warp] = (double)sm;
                }
                if (consumer_barrier_or<kConsumers>(!ok || *abortp != 0)) {
                    ok = false;
                    break;
                }
                if (warp == 0) {  // one lane per warp's partial: the rescaling exponentials run side by side
                    const float wmx = lane < kConsumerWarps ? sh_m[lane] : -INFINITY;
                    const double wsum = lane < kConsumerWarps ? sh_s[lane] : 0.0;
                    const float mm = warp_max(wmx);
                    double tot = (wsum > 0.0) ? wsum * exp((double)wmx - (double)mm) : 0.0;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
                    if (lane == 0) {
                        const double lse = (double)mm + log(tot);
                        sh_lse = lse;
                        sh_M = mm;
                        ws.row_state[r] = ROW_OK;
                        ws.lse[r] = lse;
                        ws.token_logp[r] = (double)sh_zy - lse;
                        ws.row_max[r] = mm;
                    }
                }
                consumer_barrier();
            }
            if (plan != ROWS_BOTH) {
                zero_row();
                continue;
            }
            // ---- sweep 2: dlogits, in place in the warp's slice of the stage, out by the warp's own
            // bulk store ----
            const int n = (int)(r / seq_len);
            const double g = ws.coef[n];
            RowConst rc;
            if constexpr (DT == RAPID_BF16) {
                rc.c = (float)fma(-sh_lse, kLog2eD, ws.coef_log2[n]);
                rc.g = (float)g;
                rc.sign2 = (g < 0.0) ? 0x80008000u : 0u;
                rc.y = y;
            } else {
                rc.M = sh_M;
                rc.a = (float)(sh_lse - (double)sh_M);
                rc.g = (float)g;
                rc.y = y;
            }
            // chunk c of the row sits in stage s: dlogits in place, then out
            auto second_sweep_chunk = [&](int c, int s) {
                uint4* sv = reinterpret_cast<uint4*>(ring + (size_t)s * kChunk);
                const int v0 = c * kVecPerChunk;
                const int nv = min(kVecPerChunk, nvec_row - v0);
                if (c == n_chunks - 1) {
                    const int e = nvec_row * PER + tid;
                    if (e < vocab) dz_scalar(sv, orow, e - v0 * PER, e, rc);
                }
                uint4* wv = sv + warp * kVecPerWarp + lane;
                const int nvw = nv - warp * kVecPerWarp;  // whole vectors in this warp's slice
                const int e0 = (v0 + warp * kVecPerWarp + lane) * PER;  // first column of this thread's first vector
                if (nvw >= kVecPerWarp) {
                    uint4 z[kVecPerThread];
#pragma unroll
                    for (int j = 0; j < kVecPerThread; ++j) z[j] = wv[j * 32];
#pragma unroll
                    for (int j = 0; j < kVecPerThread; ++j) {
                        const int e = e0 + j * 32 * PER;
                        // the sampled token's column is looked for once per vector, not once per element
                        wv[j * 32] = dz_vec_any(z[j], e, rc);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < kVecPerThread; ++j)
                        if (j * 32 + lane < nvw) wv[j * 32] = dz_vec<true>(wv[j * 32], e0 + j * 32 * PER, rc);
                }
                fence_proxy_async_smem();  // generic writes above -> asynchronous read below
                __syncwarp();
                if (lane == 0) {
                    if (nvw > 0) {
                        const size_t off = (size_t)warp * kVecPerWarp * 16;
                        bulk_store_hint(orow + (size_t)c * kChunk + off, reinterpret_cast<uint8_t*>(sv) + off,
                                        (uint32_t)min(nvw, kVecPerWarp) * 16u, stream);
                        bulk_commit();
                        pushed(s);
                    } else {
                        mbar_arrive(&empty_bar[s]);  // nothing to send from this slice
                    }
                }
            };
            {   // first the chunks kept from the first sweep, where they lie
                int rs = ret_st;
                for (int c = n_chunks - n_ret; c < n_chunks; ++c) {
                    second_sweep_chunk(c, rs);
                    if (++rs == kStages) rs = 0;
                }
            }
            for (int c = 0; c < n_chunks - n_ret && ok; ++c) {
                const int s = st;
                const bool got = mbar_wait_bounded(&full_bar[s], ph, abortp);
                if (__any_sync(0xffffffffu, !got)) {
                    ok = false;
                    break;
                }
                next_stage();
                second_sweep_chunk(c, s);
            }
        }
        // a warp that gave up in the middle of a row still owes nothing to a barrier: the others see
        // the abort flag in their next wait
        if (lane == 0) bulk_wait_all<0>();
    }
    __syncthreads();
    if (tid == 0 && abort_flag) atomicMax(&ws.stats->status, (int)RAPID_ERR_TIMEOUT);
}

// ---- after the pass: the loss and the statistics ---------------------------------------------------------

__global__ void __launch_bounds__(kPrepThreads)
onpolicy_loss_kernel(int n_seq, float* __restrict__ loss_out, rapid_stats_t* __restrict__ stats_out, Workspace ws) {
    __shared__ double sh_d[kPrepThreads / 32];
    __shared__ long long sh_l[kPrepThreads / 32];
    __shared__ int sh_i[kPrepThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    double loss = 0.0;
    long long tokens = 0;
    int bad = 0;
    for (int n = tid; n < n_seq; n += kPrepThreads) {
        loss -= ws.coef[n] * ws.seq_logp[n];
        tokens += ws.seq_tokens[n];
        bad += ws.seq_bad[n];
    }
    loss = warp_sum(loss);
    tokens = warp_sum(tokens);
    bad = warp_sum(bad);
    if (lane == 0) {
        sh_d[warp] = loss;
        sh_l[warp] = tokens;
        sh_i[warp] = bad;
    }
    __syncthreads();
    if (tid == 0) {
        double L = 0.0;
        long long tk = 0;
        int bd = 0;
        for (int w = 0; w < kPrepThreads / 32; ++w) {
            L += sh_d[w];
            tk += sh_l[w];
            bd += sh_i[w];
        }
        rapid_stats_t st;
        st.status = ws.stats->status;
        st.n_empty_group = ws.stats->n_empty_group;
        if (st.status == RAPID_ERR_INVALID_ARG) L = (double)__int_as_float(0x7fc00000);
        st.n_tokens = tk;
        st.n_clipped = 0;       // every weight is exactly 1
        st.n_bad_token = bd;
        st.mean_log_cw = 0.0;
        st.mean_abs_log_cw = 0.0;
        st.loss = L;
        *ws.stats = st;
        if (stats_out) *stats_out = st;
        if (loss_out) *loss_out = (float)L;
    }
}

}  // namespace

cudaError_t launch_onpolicy(const rapid_desc_t& d, const void* logits, void* dlogits, const int32_t* targets,
                            const uint8_t* mask, const float* rewards, const int32_t* group_offsets, float* loss,
                            float* token_logp, float* adv, rapid_stats_t* stats, const Workspace& ws, int sm_count,
                            cudaStream_t stream) {
    const int64_t T = (int64_t)d.n_seq * d.seq_len;
    onpolicy_prep_kernel<<<1, kPrepThreads, 0, stream>>>(d.n_seq, d.seq_len, d.vocab, d.n_groups, d.norm_z, d.flags,
                                                        rewards, group_offsets, targets, mask, adv, ws);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    constexpr size_t smem = (size_t)kStages * kChunk + kZeroBuf;
    const int want_logp = token_logp != nullptr;
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        int per_sm = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, smem);
        if (err != cudaSuccess) return err;
        if (per_sm < 1) per_sm = 1;
        int64_t grid = (int64_t)sm_count * per_sm;
        if (grid > T) grid = T;
        if (T > 0xffffffffll) return cudaErrorInvalidValue;  // the row counter is 32 bits wide
        err = cudaMemsetAsync(ws.row_ticket, 0, 2 * sizeof(unsigned int), stream);
        if (err != cudaSuccess) return err;
#ifndef RAPID_OP_FILL_FIRST
#define RAPID_OP_FILL_FIRST 0  // measured: 5.73 ms with the fills first against 5.56-5.64 interleaved (the live rows of this kernel are not HBM-bound, so the fills overlap them for free)
#endif
        const int fill_first = RAPID_OP_FILL_FIRST && (double)T * (double)d.vocab * (d.dtype == RAPID_BF16 ? 2.0 : 4.0) >= 8.0e9;
        kern<<<(unsigned)grid, kThreads, smem, stream>>>(logits, dlogits, d.ld, d.vocab, d.seq_len, T, targets, mask,
                                                         want_logp, ws.row_ticket, scatter_stride(T), fill_first, ws);
        return cudaGetLastError();
    };
    e = (d.dtype == RAPID_BF16) ? go(onpolicy_rows_kernel<RAPID_BF16>) : go(onpolicy_rows_kernel<RAPID_F32>);
    if (e != cudaSuccess) return e;
    e = launch_seq_reduce(d, nullptr, token_logp, ws, stream);
    if (e != cudaSuccess) return e;
    onpolicy_loss_kernel<<<1, kPrepThreads, 0, stream>>>(d.n_seq, loss, stats, ws);
    return cudaGetLastError();
}

}  // namespace rapid
