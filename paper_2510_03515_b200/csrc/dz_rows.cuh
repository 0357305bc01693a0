// dlogits of one row from its logits, shared by the second pass of the two-pass path and the second
// sweep of the on-policy kernel:
//     dz[v] = g (softmax(z)_v - 1[v == y]),   softmax(z)_v = exp(z_v - lse)
// (the derivative of the Eq. 3 surrogate through the log-softmax, for one unmasked token).
//
// bf16: g is folded into the exponent, dz = sign(g) 2^(z log2(e) - lse log2(e) + log2|g|), so an
// element costs one fused multiply-add and one MUFU exponential.
// fp32: p = exp((z - M) - (lse - M)) with the accurate exponential, then times g.
#pragma once

#include "rapid_common.cuh"

#ifndef RAPID_DZ_F32X2
#define RAPID_DZ_F32X2 1  // packed two-float arithmetic in the bf16 form
#endif

namespace rapid {

struct RowConstBf16 {
    float c;         // -lse log2(e) + log2|g|
    float g;         // coefficient
    uint32_t sign2;  // sign of g on both halves of a packed pair
    int y;           // sampled token
};
struct RowConstF32 {
    float M, a, g;  // row max, lse - M, coefficient
    int y;
};

__device__ __forceinline__ uint16_t float_to_bf16_bits(float x) { return (uint16_t)(pack_bf16x2(x, 0.f) & 0xffffu); }

// One 16-byte vector of logits -> dlogits; `e0` is the column of its first element.  HAS_Y says
// whether the sampled token's column may lie in this vector (the caller tests that once per vector).
template <bool HAS_Y>
__device__ __forceinline__ uint4 dz_vec(uint4 z, int e0, const RowConstBf16& rc) {
    uint32_t w[4] = {z.x, z.y, z.z, z.w};
#if RAPID_DZ_F32X2
    const uint64_t k2 = f32x2(kLog2e, kLog2e), c2 = f32x2(rc.c, rc.c);
#endif
#pragma unroll
    for (int k = 0; k < 4; ++k) {
#if RAPID_DZ_F32X2
        float xl, xh;
        f32x2_split(f32x2_fma(f32x2(bf16_lo(w[k]), bf16_hi(w[k])), k2, c2), xl, xh);
        const float lo = ex2_approx(xl), hi = ex2_approx(xh);
#else
        const float lo = ex2_approx(fmaf(bf16_lo(w[k]), kLog2e, rc.c));
        const float hi = ex2_approx(fmaf(bf16_hi(w[k]), kLog2e, rc.c));
#endif
        uint32_t out = pack_bf16x2(lo, hi) ^ rc.sign2;
        if (HAS_Y && e0 + 2 * k == (rc.y & ~1)) {  // the sampled token: g (p_y - 1), formed in float before rounding
            const float ps = (rc.y & 1) ? hi : lo;
            const uint32_t b = float_to_bf16_bits((rc.g < 0.f ? -ps : ps) - rc.g);
            out = (rc.y & 1) ? ((out & 0x0000ffffu) | (b << 16)) : ((out & 0xffff0000u) | b);
        }
        w[k] = out;
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}
template <bool HAS_Y>
__device__ __forceinline__ uint4 dz_vec(uint4 zb, int e0, const RowConstF32& rc) {
    const float z[4] = {__uint_as_float(zb.x), __uint_as_float(zb.y), __uint_as_float(zb.z), __uint_as_float(zb.w)};
    uint32_t o[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        float v = rc.g * expf((z[k] - rc.M) - rc.a);
        if (HAS_Y && e0 + k == rc.y) v -= rc.g;
        o[k] = __float_as_uint(v);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// The same with the test for the sampled token's column made here, once for the vector.
template <class RowConst>
__device__ __forceinline__ uint4 dz_vec_any(uint4 z, int e0, const RowConst& rc) {
    constexpr int PER = std::is_same<RowConst, RowConstBf16>::value ? 8 : 4;
    return ((unsigned)(rc.y - e0) < (unsigned)PER) ? dz_vec<true>(z, e0, rc) : dz_vec<false>(z, e0, rc);
}

// scalar tail elements (vocab not a multiple of the vector width): read from the stage in shared
// memory, written straight to global memory
__device__ __forceinline__ void dz_scalar(const void* zsm, void* orow, int e_in_chunk, int e, const RowConstBf16& rc) {
    const float z = __uint_as_float(((uint32_t) static_cast<const uint16_t*>(zsm)[e_in_chunk]) << 16);
    const float ps = ex2_approx(fmaf(z, kLog2e, rc.c));
    float val = (rc.g < 0.f) ? -ps : ps;
    if (e == rc.y) val -= rc.g;
    static_cast<uint16_t*>(orow)[e] = float_to_bf16_bits(val);
}
__device__ __forceinline__ void dz_scalar(const void* zsm, void* orow, int e_in_chunk, int e, const RowConstF32& rc) {
    const float z = static_cast<const float*>(zsm)[e_in_chunk];
    float val = rc.g * expf((z - rc.M) - rc.a);
    if (e == rc.y) val -= rc.g;
    static_cast<float*>(orow)[e] = val;
}

// Named barrier 1 over the first N threads of the CTA (the consumer warps), returning the OR of
// `flag` over all of them: the decision to leave after a timeout is taken by everyone together, so
// nobody is left waiting at a later barrier.
template <int N>
__device__ __forceinline__ bool consumer_barrier_or(bool flag) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"((uint32_t)flag), "n"(N)
        : "memory");
    return out != 0;
}

}  // namespace rapid
