// Pass 2: re-read the logits once and write
//     dlogits[r, v] = g_n m_r (softmax(z[r, .])_v - 1[v == y_r]),
// the derivative of the Eq. 3 surrogate loss through the log-softmax.  Rows that are masked or
// whose coefficient g_n is zero are written as zeros without reading the logits.  Each thread
// reads a 16-byte vector and writes the same 16 bytes, so dlogits may be the logits buffer.
//
// bf16: g_n is folded into the exponent, dz = sign(g) 2^(z log2(e) - lse log2(e) + log2|g|), so the
// inner loop is one fused multiply-add and one MUFU exponential per element.
// fp32: p = exp((z - M) - (lse - M)) with the accurate exponential, then times g.
#include "rapid_common.cuh"

namespace rapid {

namespace {

constexpr int kThreads = 256;

template <int U>
__device__ __forceinline__ void dz_batch_bf16(uint4 (&q)[U], float c, uint32_t sign2) {
#pragma unroll
    for (int j = 0; j < U; ++j) {
        uint32_t w[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float lo = ex2_approx(fmaf(bf16_lo(w[k]), kLog2e, c));
            const float hi = ex2_approx(fmaf(bf16_hi(w[k]), kLog2e, c));
            w[k] = pack_bf16x2(lo, hi) ^ sign2;
        }
        q[j] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

__device__ __forceinline__ uint16_t float_to_bf16_bits(float x) {
    return (uint16_t)(pack_bf16x2(x, 0.f) & 0xffffu);
}

// one row, bf16
__device__ __forceinline__ void dz_row_bf16(const uint16_t* zrow, uint16_t* orow, int vocab, int y,
                                            float c, float g) {
    constexpr int U = 4;
    const int tid = threadIdx.x;
    const int nvec = vocab >> 3;
    const uint4* rv = reinterpret_cast<const uint4*>(zrow);
    uint4* ov = reinterpret_cast<uint4*>(orow);
    const uint32_t sign2 = (g < 0.f) ? 0x80008000u : 0u;
    const int yv = y >> 3;

    auto fix_target = [&](uint4& q, const uint4& zq) {
        // the sampled token's entry is g (p_y - 1): recompute it in float from the logit
        const uint32_t zw[4] = {zq.x, zq.y, zq.z, zq.w};
        uint32_t ow[4] = {q.x, q.y, q.z, q.w};
        const int k = (y & 7) >> 1;
        const bool hi = (y & 1) != 0;
        const float z = hi ? bf16_hi(zw[k]) : bf16_lo(zw[k]);
        const float p_scaled = ex2_approx(fmaf(z, kLog2e, c));  // |g| p_y
        const float val = (g < 0.f ? -p_scaled : p_scaled) - g;
        const uint32_t b = float_to_bf16_bits(val);
        ow[k] = hi ? ((ow[k] & 0x0000ffffu) | (b << 16)) : ((ow[k] & 0xffff0000u) | b);
        q = make_uint4(ow[0], ow[1], ow[2], ow[3]);
    };

    int v = tid;
    for (; v + (U - 1) * kThreads < nvec; v += U * kThreads) {
        uint4 z[U], q[U];
#pragma unroll
        for (int j = 0; j < U; ++j) q[j] = z[j] = ld_stream(rv + v + j * kThreads);
        dz_batch_bf16<U>(q, c, sign2);
#pragma unroll
        for (int j = 0; j < U; ++j) {
            if (v + j * kThreads == yv) fix_target(q[j], z[j]);
            st_stream(ov + v + j * kThreads, q[j]);
        }
    }
    for (; v < nvec; v += kThreads) {
        uint4 z[1], q[1];
        q[0] = z[0] = ld_stream(rv + v);
        dz_batch_bf16<1>(q, c, sign2);
        if (v == yv) fix_target(q[0], z[0]);
        st_stream(ov + v, q[0]);
    }
    const int e = (nvec << 3) + tid;
    if (e < vocab) {
        const float z = __uint_as_float(((uint32_t)zrow[e]) << 16);
        const float ps = ex2_approx(fmaf(z, kLog2e, c));
        float val = (g < 0.f) ? -ps : ps;
        if (e == y) val -= g;
        orow[e] = float_to_bf16_bits(val);
    }
}

// one row, fp32
__device__ __forceinline__ void dz_row_f32(const float* zrow, float* orow, int vocab, int y, float M,
                                           float a, float g) {
    constexpr int U = 4;
    const int tid = threadIdx.x;
    const int nvec = vocab >> 2;
    const float4* rv = reinterpret_cast<const float4*>(zrow);
    float4* ov = reinterpret_cast<float4*>(orow);
    const int yv = y >> 2;
    auto one = [&](float z) { return g * expf((z - M) - a); };
    auto vec = [&](float4 z, int vi) {
        float4 o = make_float4(one(z.x), one(z.y), one(z.z), one(z.w));
        if (vi == yv) {
            const int k = y & 3;
            if (k == 0) o.x -= g;
            else if (k == 1) o.y -= g;
            else if (k == 2) o.z -= g;
            else o.w -= g;
        }
        return o;
    };
    int v = tid;
    for (; v + (U - 1) * kThreads < nvec; v += U * kThreads) {
        float4 z[U];
#pragma unroll
        for (int j = 0; j < U; ++j) z[j] = __ldcs(rv + v + j * kThreads);
#pragma unroll
        for (int j = 0; j < U; ++j) __stcs(ov + v + j * kThreads, vec(z[j], v + j * kThreads));
    }
    for (; v < nvec; v += kThreads) __stcs(ov + v, vec(__ldcs(rv + v), v));
    const int e = (nvec << 2) + tid;
    if (e < vocab) {
        float val = one(zrow[e]);
        if (e == y) val -= g;
        orow[e] = val;
    }
}

template <int ESIZE>
__device__ __forceinline__ void zero_row(void* orow, int vocab) {
    const int tid = threadIdx.x;
    constexpr int per = 16 / ESIZE;
    const int nvec = vocab / per;
    uint4* ov = reinterpret_cast<uint4*>(orow);
    for (int v = tid; v < nvec; v += kThreads) st_stream(ov + v, make_uint4(0, 0, 0, 0));
    const int e = nvec * per + tid;
    if (e < vocab) {
        if (ESIZE == 2) static_cast<uint16_t*>(orow)[e] = 0;
        else static_cast<float*>(orow)[e] = 0.f;
    }
}

template <int DT>
__global__ void __launch_bounds__(kThreads)
dlogits_kernel(const void* logits, void* dlogits /* may alias logits */, int64_t ld, int vocab,
               int seq_len, int64_t row0, int64_t n_rows, const int32_t* __restrict__ targets,
               Workspace ws) {
    for (int64_t i = blockIdx.x; i < n_rows; i += gridDim.x) {
        const int64_t r = row0 + i;
        const int n = (int)(r / seq_len);
        const double g = ws.coef[n];
        const bool live = (ws.row_state[r] == ROW_OK) && (g != 0.0);
        if (DT == RAPID_BF16) {
            uint16_t* orow = static_cast<uint16_t*>(dlogits) + i * ld;
            if (!live) {
                zero_row<2>(orow, vocab);
                continue;
            }
            const float c = (float)fma(-ws.lse[r], kLog2eD, ws.coef_log2[n]);
            dz_row_bf16(static_cast<const uint16_t*>(logits) + i * ld, orow, vocab, targets[r], c,
                        (float)g);
        } else {
            float* orow = static_cast<float*>(dlogits) + i * ld;
            if (!live) {
                zero_row<4>(orow, vocab);
                continue;
            }
            const float M = ws.row_max[r];
            const float a = (float)(ws.lse[r] - (double)M);
            dz_row_f32(static_cast<const float*>(logits) + i * ld, orow, vocab, targets[r], M, a,
                       (float)g);
        }
    }
}

}  // namespace

cudaError_t launch_dlogits(const rapid_desc_t& d, const void* logits_chunk, void* dlogits_chunk,
                           int64_t row0, int64_t n_rows, const int32_t* targets,
                           const Workspace& ws, int sm_count, cudaStream_t stream) {
    if (n_rows <= 0) return cudaSuccess;
    int per_sm = 0;
    cudaError_t e;
    if (d.dtype == RAPID_BF16)
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dlogits_kernel<RAPID_BF16>,
                                                          kThreads, 0);
    else
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dlogits_kernel<RAPID_F32>,
                                                          kThreads, 0);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    int64_t grid = (int64_t)sm_count * per_sm;
    if (grid > n_rows) grid = n_rows;
    if (d.dtype == RAPID_BF16)
        dlogits_kernel<RAPID_BF16><<<(unsigned)grid, kThreads, 0, stream>>>(
            logits_chunk, dlogits_chunk, d.ld, d.vocab, d.seq_len, row0, n_rows, targets, ws);
    else
        dlogits_kernel<RAPID_F32><<<(unsigned)grid, kThreads, 0, stream>>>(
            logits_chunk, dlogits_chunk, d.ld, d.vocab, d.seq_len, row0, n_rows, targets, ws);
    return cudaGetLastError();
}

}  // namespace rapid
