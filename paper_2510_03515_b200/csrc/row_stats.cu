// Pass 1: per-row log-sum-exp over the vocabulary and the sampled token's log-probability
// (the softmax policy's log pi_theta(y_t|.), the quantity that Eq. 3 and Eq. 5 are built from).
//
// One CTA streams one row at a time with 128-bit loads; rows are taken grid-stride.  Masked rows
// and rows with an invalid token id are not read.
//
// bf16 logits: one sweep, online max/sum per thread in float (base-2 exponentials on the MUFU
// pipe), combined across the CTA in double.
// fp32 logits: also one sweep, with the accurate exponential; the tolerance on the loss is tight (a
// generation sums thousands of token log-probs), so threads are combined in double.
#include "rapid_common.cuh"

namespace rapid {

namespace {

#ifndef RAPID_P1_THREADS
#define RAPID_P1_THREADS 128  // bf16 logits
#endif
#ifndef RAPID_P1_THREADS_F32
#define RAPID_P1_THREADS_F32 128  // float logits
#endif
#ifndef RAPID_P1_U
#define RAPID_P1_U 8  // 16-byte loads in flight per thread (bf16 sweep)
#endif
#ifndef RAPID_P1_TICKETS
#define RAPID_P1_TICKETS 1  // rows handed out through a counter (1) or grid-stride (0)
#endif

// ---- bf16 ------------------------------------------------------------------------------------

// One batch of U vectors: the batch's exponentials are summed in float from zero and then added to
// the thread's running sum with an error-compensated add (the rounding error of every add is kept in
// a second float and folded back in at the end).  A plain float running sum silently drops terms
// below half an ulp of the sum -- with a peaked softmax that is most of the tail -- and the lost mass
// shows up as a bias of a few 1e-7 per token log-prob, which a generation-level weight then
// multiplies by its length.  (A double running sum does the same job but costs 2-3 % on this part's
// slow double-precision pipe.)
struct FloatSum {
    float s, c;  // running sum and the accumulated rounding error of its adds
    __device__ __forceinline__ void add(float x) {  // requires s >= x >= 0 or s == 0: Fast2Sum
        const float t = s + x;
        c += (s - t) + x;
        s = t;
    }
    __device__ __forceinline__ void scale(float f) {
        s *= f;
        c *= f;
    }
    __device__ __forceinline__ double value() const { return (double)s + (double)c; }
};

// A thread's state is (m, sh, S): the largest logit seen, the shift sh that its exponentials were taken
// against, and S = sum_v 2^(x_v) with x_v = z_v log2(e) - sh.  A generation-level weight multiplies
// any bias of the token log-probs by the generation's length, so four things keep the log-sum-exp
// free of bias beyond about 1e-9:
//  * sh = ceil(m log2 e) + off is USED as it stands, in the exponentials and again when threads are
//    combined (in double), so no rounding of m log2(e) enters.  Its integer part makes moving to a new
//    shift a multiplication by an exact power of two.
//  * log2(e) is applied as kK1 + kK2: kK1 has 16 significant bits, so its product with a bf16 logit
//    (8 bits) is exact, and the float kK2 carries the next 24 bits.  A single float constant is off by
//    1.3e-8 relative, which shifts the log-sum-exp by that times the softmax-weighted mean distance
//    below the shift: 5e-8 for these logits.
//  * the hardware exponential's relative error on negative arguments, averaged over the fraction of
//    the argument, is kEx2Bias (measured over all 2^23 fractions on sm_100a: -4.95e-8 for arguments in
//    [-1, 0), -4.97e-8 in [-2, -1), -5.02e-8 in [-5, -4), -5.11e-8 in [-20, -19); the terms that carry a
//    row's mass lie within a few units of the shift; errors lie in [-1.44e-7, +0.63e-7]); a sum of many
//    terms carries that mean, and is divided by 1 + kEx2Bias.  bf16 logits take few distinct values, so with a common
//    integer shift the fraction of x_v would depend on z_v alone and the sum would carry the errors of
//    those few fractions (1e-8 either way) instead of the mean; the 16-bit fraction `off`, different
//    for every thread, spreads each logit value over 128 fractions.
//  * the thread's largest logit, which may carry nearly all of the row's probability, gets no such
//    statistical treatment: its hardware exponential is taken out of S again at the end of the sweep
//    and replaced by the exact value in double.
constexpr float kEx2Bias = -4.95e-8f;
constexpr float kK1 = 47274.f / 32768.f;                   // log2(e) rounded down to 16 bits
constexpr float kK2 = (float)(kLog2eD - 47274.0 / 32768.0);  // > 0, so that -inf logits stay -inf

template <int U>
__device__ __forceinline__ void bf16_batch(const uint4 (&q)[U], float off, float& m, float& sh, FloatSum& S) {
    uint32_t mx = bf16x2_max(bf16x2_max(q[0].x, q[0].y), bf16x2_max(q[0].z, q[0].w));
#pragma unroll
    for (int j = 1; j < U; ++j)
        mx = bf16x2_max(mx, bf16x2_max(bf16x2_max(q[j].x, q[j].y), bf16x2_max(q[j].z, q[j].w)));
    const float bm = fmaxf(bf16_lo(mx), bf16_hi(mx));
    // logits may be -inf or the lowest finite value (a masked part of the vocabulary): while the thread
    // has seen nothing else it keeps the shift 0, so that the shift neither turns (-inf) - (-inf) into
    // a NaN nor overflows to +inf
    if (bm > m) {  // rare after the first few batches
        m = bm;
        if (bm > -1.0e38f) {
            const float nsh = ceilf(bm * kLog2e) + off;
            S.scale(ex2_approx(sh - nsh));  // an exact power of two (S is still 0 for an empty thread's shift 0)
            sh = nsh;
        }
    }
    // a pair of logits at a time in the packed two-float forms (one instruction for two multiply-adds
    // or two additions, each rounded like its scalar form)
    const uint64_t k1 = f32x2(kK1, kK1), k2 = f32x2(kK2, kK2), nsh2 = f32x2(-sh, -sh);
    // eight partial sums of at most U terms each (four packed pairs, one per word of a vector): a float
    // partial that holds one of the row's largest terms drops every later addend below half an ulp of
    // it, and the fewer addends share a partial with such a term, the less is lost (with two partials of
    // 32 terms that loss was the largest bias left, 2e-9 on N(0,3) logits)
    uint64_t s2[4] = {f32x2(0.f, 0.f), f32x2(0.f, 0.f), f32x2(0.f, 0.f), f32x2(0.f, 0.f)};
#pragma unroll
    for (int j = 0; j < U; ++j) {
        const uint32_t w[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint64_t z2 = f32x2(bf16_lo(w[k]), bf16_hi(w[k]));
            float x0, x1;
            f32x2_split(f32x2_fma(z2, k2, f32x2_fma(z2, k1, nsh2)), x0, x1);
            s2[k] = f32x2_add(s2[k], f32x2(ex2_approx(x0), ex2_approx(x1)));
        }
    }
    float s0, s1;
    f32x2_split(f32x2_add(f32x2_add(s2[0], s2[1]), f32x2_add(s2[2], s2[3])), s0, s1);
    const float b = s0 + s1;
    if (b > S.s) {  // keep the larger operand first, as Fast2Sum wants (early batches only)
        const float old = S.s;
        S.s = b;
        S.add(old);
    } else {
        S.add(b);
    }
}

// `out`, when not null, receives a copy of the row (same layout): used when the logits are read from
// host memory and the second pass wants them on the device.
// Returns the thread's maximum, its shift (log2 units) and its share of sum_v 2^(z_v log2(e) - sh), all
// corrections applied; a thread that saw nothing real returns 0 and the shift 0.
template <int kThreads>
__device__ __forceinline__ void row_sweep_bf16(const uint16_t* row, int vocab, float& m_out, float& sh_out,
                                               double& s_out, uint16_t* out) {
    constexpr int U = RAPID_P1_U;
    const int tid = threadIdx.x;
    const int nvec = vocab >> 3;
    const uint4* rv = reinterpret_cast<const uint4*>(row);
    uint4* ov = reinterpret_cast<uint4*>(out);
    float m = -INFINITY, sh = 0.f;
    FloatSum S{0.f, 0.f};
    // this thread's fraction of the shift (see above): 16 bits, scattered, so that the fractions neither
    // line up with a table of the hardware exponential nor cost the shift its exactness
    const float off = (float)(((unsigned)tid * 40503u) & 0xffffu) * (1.f / 65536.f);
    int v = tid;
    for (; v + (U - 1) * kThreads < nvec; v += U * kThreads) {
        uint4 q[U];
#pragma unroll
        for (int j = 0; j < U; ++j) q[j] = ld_stream(rv + v + j * kThreads);
        if (out) {
#pragma unroll
            for (int j = 0; j < U; ++j) ov[v + j * kThreads] = q[j];
        }
        bf16_batch<U>(q, off, m, sh, S);
    }
    for (; v < nvec; v += kThreads) {
        uint4 q[1];
        q[0] = ld_stream(rv + v);
        if (out) ov[v] = q[0];
        bf16_batch<1>(q, off, m, sh, S);
    }
    // ragged tail (vocab not a multiple of 8): one element per thread
    double tail = 0.0;
    const int e = (nvec << 3) + tid;
    if (e < vocab) {
        const uint16_t zb = row[e];
        if (out) out[e] = zb;
        const float z = __uint_as_float(((uint32_t)zb) << 16);
        if (z > m) {
            m = z;
            if (z > -1.0e38f) {
                const float nsh = ceilf(z * kLog2e) + off;
                S.scale(ex2_approx(sh - nsh));
                sh = nsh;
            }
        }
        if (z > -1.0e38f) tail = (double)ex2_approx(fmaf(z, kK2, fmaf(z, kK1, -sh)));
    }
    m_out = m;
    sh_out = sh;
    double s = S.value() + tail, top = 0.0;
    if (m > -1.0e38f) {  // the largest logit: out with what the hardware gave for it, in with the exact term
        s -= (double)ex2_approx(fmaf(m, kK2, fmaf(m, kK1, -sh)));
        top = exp2((double)m * kLog2eD - (double)sh);
    }
    s_out = s / (1.0 + (double)kEx2Bias) + top;
}

// ---- fp32 ------------------------------------------------------------------------------------

// One sweep, online: every thread keeps its own running maximum and the sum of accurate
// exponentials against it, four at a time in float and accumulated in double (rescaled in double on
// the rare occasions the maximum moves); threads are combined in double afterwards.  A generation's
// weight sums thousands of token log-probs, so a bias of even 1e-8 per row would show.
__device__ __forceinline__ void f32_batch(const float4* q, int n, float& m, double& s) {
    float bm = -INFINITY;
    for (int j = 0; j < n; ++j) bm = fmaxf(bm, fmaxf(fmaxf(q[j].x, q[j].y), fmaxf(q[j].z, q[j].w)));
    if (bm > m) {
        if (s > 0.0) s *= exp((double)m - (double)bm);
        m = bm;
    }
    if (m == -INFINITY) return;  // nothing but -inf so far (a masked part of the vocabulary): the sum stays 0
    for (int j = 0; j < n; ++j)
        s += (double)((expf(q[j].x - m) + expf(q[j].y - m)) + (expf(q[j].z - m) + expf(q[j].w - m)));
}

template <int kThreads>
__device__ __forceinline__ void row_sweep_f32(const float* row, int vocab, float& m_out, double& s_out,
                                              float* out) {
    constexpr int U = 4;
    const int tid = threadIdx.x;
    const int nvec = vocab >> 2;
    const float4* rv = reinterpret_cast<const float4*>(row);
    float4* ov = reinterpret_cast<float4*>(out);
    float m = -INFINITY;
    double s = 0.0;
    int v = tid;
    for (; v + (U - 1) * kThreads < nvec; v += U * kThreads) {
        float4 q[U];
#pragma unroll
        for (int j = 0; j < U; ++j) q[j] = __ldcs(rv + v + j * kThreads);
        if (out) {
#pragma unroll
            for (int j = 0; j < U; ++j) ov[v + j * kThreads] = q[j];
        }
        f32_batch(q, U, m, s);
    }
    for (; v < nvec; v += kThreads) {
        float4 q[1];
        q[0] = __ldcs(rv + v);
        if (out) ov[v] = q[0];
        f32_batch(q, 1, m, s);
    }
    const int e = (nvec << 2) + tid;  // ragged tail (vocab not a multiple of 4)
    if (e < vocab) {
        const float z = __ldg(row + e);
        if (out) out[e] = z;
        if (z > m) {
            if (s > 0.0) s *= exp((double)m - (double)z);
            m = z;
        }
        if (z != -INFINITY) s += (double)expf(z - m);
    }
    m_out = m;
    s_out = s;
}

// ---- kernel ----------------------------------------------------------------------------------

// Rows are handed out one at a time through a counter (`ticket`, zero at launch) when one is given, so
// that every CTA stays busy until the rows run out whatever the pattern of masked rows; without a counter
// CTA b takes rows b, b + grid, ...
template <int DT, int kThreads>
__global__ void __launch_bounds__(kThreads)
row_stats_kernel(const void* __restrict__ logits, void* __restrict__ copy_out, int64_t ld, int vocab, int64_t row0,
                 int64_t n_rows, const int32_t* __restrict__ targets,
                 const uint8_t* __restrict__ mask, unsigned int* ticket, Workspace ws) {
    constexpr int kWarps = kThreads / 32;
    __shared__ float sh_m[kWarps];
    __shared__ float sh_sh[kWarps];
    __shared__ double sh_s[kWarps];
    __shared__ unsigned int sh_next;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int64_t i = blockIdx.x;; i += gridDim.x) {
        if (ticket) {  // uniform
            if (tid == 0) sh_next = atomicAdd(ticket, 1u);
            __syncthreads();
            i = sh_next;
            __syncthreads();  // everyone has read it before thread 0 draws again
        }
        if (i >= n_rows) break;
        const int64_t r = row0 + i;
        const bool on = mask ? (mask[r] != 0) : true;
        const int32_t y = targets[r];
        if (!on || y < 0 || y >= vocab) {  // uniform across the CTA
            if (tid == 0) {
                ws.row_state[r] = on ? ROW_BAD_TOKEN : ROW_MASKED;
                ws.lse[r] = 0.0;
                ws.token_logp[r] = 0.0;
                ws.row_max[r] = 0.f;
            }
            continue;
        }

        float M;
        double S;      // the row's sum of exponentials against `shift`
        double shift;  // M for float logits; the shift actually used, in natural-log units, for bf16
        double zy;
        if (DT == RAPID_BF16) {
            const uint16_t* row = static_cast<const uint16_t*>(logits) + i * ld;
            float m, sh;
            double s;
            uint16_t* orow = copy_out ? static_cast<uint16_t*>(copy_out) + i * ld : nullptr;
            row_sweep_bf16<kThreads>(row, vocab, m, sh, s, orow);
            // threads are brought to a common shift in double, with the shifts exactly as they were used;
            // a thread (or a whole warp, for a tiny vocabulary) that saw nothing has s = 0
            const float wm = warp_max(m);
            const float wsh = warp_max(s > 0.0 ? sh : -INFINITY);
            if (s > 0.0 && sh != wsh) s *= exp2((double)sh - (double)wsh);
            s = warp_sum(s);
            if (lane == 0) {
                sh_m[warp] = wm;
                sh_sh[warp] = wsh;
                sh_s[warp] = s;
            }
            __syncthreads();
            if (tid == 0) {
                float mm = sh_m[0], msh = sh_sh[0];
                for (int w = 1; w < kWarps; ++w) {
                    mm = fmaxf(mm, sh_m[w]);
                    msh = fmaxf(msh, sh_sh[w]);
                }
                double tot = 0.0;
                for (int w = 0; w < kWarps; ++w)
                    if (sh_s[w] > 0.0) tot += sh_s[w] * exp2((double)sh_sh[w] - (double)msh);
                M = mm;
                S = tot;
                shift = (double)msh * kLn2D;  // lse = shift + log(S)
                zy = (double)__uint_as_float(((uint32_t)row[y]) << 16);  // (one more 2-byte read of the row)
            }
        } else {
            const float* row = static_cast<const float*>(logits) + i * ld;
            float m;
            double s;
            float* orow = copy_out ? static_cast<float*>(copy_out) + i * ld : nullptr;
            row_sweep_f32<kThreads>(row, vocab, m, s, orow);
            const float wm = warp_max(m);
            // a thread that saw nothing has m = -inf and s = 0
            double sd = (s > 0.0) ? s * exp((double)m - (double)wm) : 0.0;
            sd = warp_sum(sd);
            if (lane == 0) {
                sh_m[warp] = wm;
                sh_s[warp] = sd;
            }
            __syncthreads();
            if (tid == 0) {
                float mm = sh_m[0];
                for (int w = 1; w < kWarps; ++w) mm = fmaxf(mm, sh_m[w]);
                double tot = 0.0;
                for (int w = 0; w < kWarps; ++w)
                    if (sh_s[w] > 0.0) tot += sh_s[w] * exp((double)sh_m[w] - (double)mm);
                M = mm;
                S = tot;
                shift = (double)mm;
                zy = (double)row[y];
            }
        }
        if (tid == 0) {
            const double lse = shift + log(S);
            ws.lse[r] = lse;
            ws.token_logp[r] = zy - lse;
            ws.row_max[r] = M;
            ws.row_state[r] = ROW_OK;
        }
        __syncthreads();  // shared scratch is reused by the next row
    }
}

}  // namespace

template <int DT, int kThreads>
static cudaError_t launch_one(const rapid_desc_t& d, const void* logits_chunk, int64_t row0, int64_t n_rows,
                              const int32_t* targets, const uint8_t* mask, const Workspace& ws, int sm_count,
                              cudaStream_t stream, void* copy_out) {
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, row_stats_kernel<DT, kThreads>, kThreads, 0);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    int64_t grid = (int64_t)sm_count * per_sm;
    if (grid > n_rows) grid = n_rows;
    unsigned int* ticket = RAPID_P1_TICKETS ? ws.row_ticket : nullptr;
    if (ticket) {
        e = cudaMemsetAsync(ticket, 0, sizeof(unsigned int), stream);
        if (e != cudaSuccess) return e;
    }
    row_stats_kernel<DT, kThreads><<<(unsigned)grid, kThreads, 0, stream>>>(logits_chunk, copy_out, d.ld, d.vocab, row0,
                                                                           n_rows, targets, mask, ticket, ws);
    return cudaGetLastError();
}

cudaError_t launch_row_stats(const rapid_desc_t& d, const void* logits_chunk, int64_t row0,
                             int64_t n_rows, const int32_t* targets, const uint8_t* mask,
                             const Workspace& ws, int sm_count, cudaStream_t stream, void* copy_out) {
    if (n_rows <= 0) return cudaSuccess;
    if (n_rows > 0xffffffffll) return cudaErrorInvalidValue;  // the row counter is 32 bits wide
    if (d.dtype == RAPID_BF16)
        return launch_one<RAPID_BF16, RAPID_P1_THREADS>(d, logits_chunk, row0, n_rows, targets, mask, ws, sm_count,
                                                        stream, copy_out);
    return launch_one<RAPID_F32, RAPID_P1_THREADS_F32>(d, logits_chunk, row0, n_rows, targets, mask, ws, sm_count,
                                                       stream, copy_out);
}

}  // namespace rapid
