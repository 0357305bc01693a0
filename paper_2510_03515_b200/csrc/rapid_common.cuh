// Shared device helpers and the workspace layout of librapid_pg (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "rapid_pg.h"

namespace rapid {

constexpr float kLog2e = 1.4426950408889634f;
constexpr double kLog2eD = 1.4426950408889634074;
constexpr double kLn2D = 0.69314718055994530942;

// Per-row state written by the statistics pass.
enum : uint8_t { ROW_MASKED = 0, ROW_OK = 1, ROW_BAD_TOKEN = 2 };

// Device pointers carved out of the caller's workspace.  Per row: 8 (lse) + 8 (log pi) +
// 4 (row max) + 1 (state) bytes; per generation: a handful of doubles.
struct Workspace {
    double* lse;            // [T] log sum_v exp z[r, v]
    double* token_logp;     // [T] z[r, y_r] - lse[r]
    float* row_max;         // [T] max_v z[r, v]
    uint8_t* row_state;     // [T] ROW_*
    double* seq_log_ratio;  // [N] s_n
    double* seq_logp;       // [N] S_n
    double* weight;         // [N] w_n
    double* clipped_w;      // [N] c_n
    double* adv;            // [N] A_n
    double* coef;           // [N] g_n
    double* coef_log2;      // [N] log2 |g_n| (-inf when g_n == 0)
    int32_t* seq_tokens;    // [N]
    int32_t* seq_bad;       // [N] rows with a target id outside [0, V)
    rapid_stats_t* stats;   // [1]
    unsigned int* row_ticket;  // [2] row counters of the streaming kernels (zeroed by each launch)
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Carve `base` (256-byte aligned).  Returns the number of bytes used.
__host__ inline size_t carve_workspace(const rapid_desc_t& d, void* base, Workspace* w) {
    const size_t T = (size_t)d.n_seq * (size_t)d.seq_len;
    const size_t N = (size_t)d.n_seq;
    size_t off = 0;
    char* p = static_cast<char*>(base);
    auto take = [&](size_t bytes) {
        char* q = p ? p + off : nullptr;
        off = align_up(off + bytes, 256);
        return q;
    };
    Workspace ws;
    ws.lse = reinterpret_cast<double*>(take(T * 8));
    ws.token_logp = reinterpret_cast<double*>(take(T * 8));
    ws.row_max = reinterpret_cast<float*>(take(T * 4));
    ws.row_state = reinterpret_cast<uint8_t*>(take(T));
    ws.seq_log_ratio = reinterpret_cast<double*>(take(N * 8));
    ws.seq_logp = reinterpret_cast<double*>(take(N * 8));
    ws.weight = reinterpret_cast<double*>(take(N * 8));
    ws.clipped_w = reinterpret_cast<double*>(take(N * 8));
    ws.adv = reinterpret_cast<double*>(take(N * 8));
    ws.coef = reinterpret_cast<double*>(take(N * 8));
    ws.coef_log2 = reinterpret_cast<double*>(take(N * 8));
    ws.seq_tokens = reinterpret_cast<int32_t*>(take(N * 4));
    ws.seq_bad = reinterpret_cast<int32_t*>(take(N * 4));
    ws.stats = reinterpret_cast<rapid_stats_t*>(take(sizeof(rapid_stats_t)));
    ws.row_ticket = reinterpret_cast<unsigned int*>(take(2 * sizeof(unsigned int)));
    if (w) *w = ws;
    return off;
}

#ifdef __CUDACC__

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// The two halves of a packed pair of bf16 values, widened exactly to float.
__device__ __forceinline__ float bf16_lo(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t p) { return __uint_as_float(p & 0xffff0000u); }

// max of two packed bf16 pairs, element-wise
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// round two floats to a packed bf16 pair (lo in the low half), round-to-nearest-even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Two floats in one 64-bit register and the packed arithmetic on them (one instruction for two
// fused multiply-adds or two additions, each rounded like its scalar form).
__device__ __forceinline__ uint64_t f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f32x2_split(uint64_t p, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
}
__device__ __forceinline__ uint64_t f32x2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t f32x2_add(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// 16-byte streaming load (read once, do not keep in L1) and store
__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) { __stcs(p, v); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ long long warp_sum(long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

#endif  // __CUDACC__

// Rows are handed to CTAs through a counter; draw t stands for row (t * stride) mod n.  The stride is coprime
// to n (every row is visited once) and near 0.62 n, so that rows drawn at about the same time lie far apart:
// the memory system then sees the batch's average mix of rows that are read and written and rows that are
// only zero-filled, rather than one kind after the other (masked rows cluster at the end of every generation).
inline unsigned long long scatter_stride(int64_t n) {
    auto gcd = [](unsigned long long a, unsigned long long b) {
        while (b) {
            const unsigned long long c = a % b;
            a = b;
            b = c;
        }
        return a;
    };
    unsigned long long s = (unsigned long long)((double)n * 0.6180339887498949);
    if (s < 1) s = 1;
    while (gcd(s, (unsigned long long)n) != 1) ++s;
    return s;
}

// Host-side launchers (each enqueues on `stream` and returns the launch status).
cudaError_t launch_row_stats(const rapid_desc_t& d, const void* logits_chunk, int64_t row0,
                             int64_t n_rows, const int32_t* targets, const uint8_t* mask,
                             const Workspace& ws, int sm_count, cudaStream_t stream,
                             void* copy_out = nullptr);
cudaError_t launch_seq_reduce(const rapid_desc_t& d, const float* behav_logp, float* token_logp_out,
                              const Workspace& ws, cudaStream_t stream);
cudaError_t launch_finalize(const rapid_desc_t& d, const float* rewards,
                            const int32_t* group_offsets, float* loss, float* adv,
                            rapid_stats_t* stats_out, const Workspace& ws, cudaStream_t stream);
cudaError_t launch_group_advantage(const rapid_desc_t& d, const float* rewards,
                                   const double* seq_log_ratio, const int32_t* group_offsets,
                                   float* adv, double* clipped_w, rapid_stats_t* stats_out,
                                   cudaStream_t stream);
cudaError_t launch_dlogits(const rapid_desc_t& d, const void* logits_chunk, void* dlogits_chunk,
                           int64_t row0, int64_t n_rows, const int32_t* targets,
                           rapid_stats_t* stats_user, const Workspace& ws, int sm_count,
                           cudaStream_t stream);

cudaError_t launch_onpolicy(const rapid_desc_t& d, const void* logits, void* dlogits, const int32_t* targets,
                            const uint8_t* mask, const float* rewards, const int32_t* group_offsets, float* loss,
                            float* token_logp, float* adv, rapid_stats_t* stats, const Workspace& ws, int sm_count,
                            cudaStream_t stream);

}  // namespace rapid
