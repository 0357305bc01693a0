// The fused LM-head form of the path: the logits z = h W are never written to memory.
//
//   forward   z tiles are formed on the tensor cores (umma_gemm.cuh); the epilogue keeps, per row
//             and per 256-column tile, the running maximum and the sum of exponentials, and picks
//             out the sampled token's logit.  A small merge kernel turns the per-tile pairs into
//             lse and log pi_theta(y_t) in double, in the same workspace layout the logits-in
//             path uses, so the per-generation reduce and the finalize step are shared.
//   backward  z tiles are formed again; the epilogue turns them into
//             dz = g_n m_r (softmax - onehot) in bf16 and stores them (TMA) into a scratch
//             matrix.  Two more GEMMs follow: dh = dz W^T (K = vocabulary) and dW = h^T dz
//             (K = rows; both operands read MN-major straight from their row-major storage).
//
// Four GEMM-sized contractions in all (forward, recompute, dh, dW); only dz, in bf16, ever
// exists in memory.
#include <math.h>

#include "rapid_common.cuh"
#include "umma_gemm.cuh"
#include "umma_gemm_pair.cuh"

namespace rapid {

namespace {

using namespace umma;

// The backward part runs over at most this many rows at a time, which bounds the dlogits scratch
// (rows x vocabulary in bf16) whatever the size of the mini-batch; dW accumulates across chunks.
constexpr int64_t kHeadChunkRows = 16384;

// Scratch of the fused-head call, carved after the ordinary workspace.
struct HeadScratch {
    float* part_m;   // [n_tiles][T] running maximum of a row within one 256-column tile
    float* part_s;   // [n_tiles][T] sum of exp(z - part_m)
    float* zy;       // [T] the sampled token's logit
    uint16_t* dz;    // [min(T, kHeadChunkRows)][ldz] bf16 ([T][ldz] when the logits are stored)
    int* status;     // raised to RAPID_ERR_TIMEOUT by a kernel whose bounded wait ran out
    int64_t ldz;
    int n_tiles;
};

inline size_t carve_head(const rapid_desc_t& d, void* base, size_t off0, HeadScratch* h) {
    const size_t T = (size_t)d.n_seq * (size_t)d.seq_len;
    const size_t nt = ((size_t)d.vocab + BN - 1) / BN;
    const size_t ldz = ((size_t)d.vocab + 63) / 64 * 64;
    size_t off = off0;
    char* p = static_cast<char*>(base);
    auto take = [&](size_t bytes) {
        char* q = p ? p + off : nullptr;
        off = align_up(off + bytes, 1024);
        return q;
    };
    HeadScratch s;
    s.part_m = reinterpret_cast<float*>(take(nt * T * 4));
    s.part_s = reinterpret_cast<float*>(take(nt * T * 4));
    s.zy = reinterpret_cast<float*>(take(T * 4));
    // with stored logits the matrix holds every row's logits first and its dlogits afterwards
    const bool store_z = (d.flags & RAPID_FLAG_HEAD_STORE_LOGITS) != 0;
    const size_t dz_rows = (store_z || T < (size_t)kHeadChunkRows) ? T : (size_t)kHeadChunkRows;
    s.dz = reinterpret_cast<uint16_t*>(take(dz_rows * ldz * 2));
    s.status = reinterpret_cast<int*>(take(256));
    s.ldz = (int64_t)ldz;
    s.n_tiles = (int)nt;
    if (h) *h = s;
    return off;
}

// ---- forward epilogue: per-tile row statistics ------------------------------------------------------

struct FwdStats {
    struct Params {
        float* part_m;
        float* part_s;
        float* zy;
        const int32_t* targets;
        int T, V;
    };
    const Params& p;
    const int row_off;  // row of this thread inside the tile
    __device__ FwdStats(const Params& p_, uint8_t*, int quarter, int lane) : p(p_), row_off(quarter * 32 + lane) {}

    __device__ void tile(int m0, int n0, uint32_t taddr) {
        const int row = m0 + row_off;
        const int ncols = min(BN, p.V - n0);
        const int ycol = (row < p.T) ? (p.targets[row] - n0) : -1;
        float m = -INFINITY, s0 = 0.f, s1 = 0.f, zyv = 0.f;
#pragma unroll 1
        for (int c = 0; c * 32 < ncols; ++c) {
            uint32_t r[32];
            tmem_ld32(taddr + c * 32, r);
            tmem_ld_wait();
            if (c * 32 + 32 > ncols) {  // ragged last chunk of the vocabulary: those columns do not exist
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (c * 32 + j >= ncols) r[j] = 0xff800000u;  // -inf
            }
            float cm = __uint_as_float(r[0]);
#pragma unroll
            for (int j = 1; j < 32; ++j) cm = fmaxf(cm, __uint_as_float(r[j]));
            if (cm > m) {
                const float f = ex2_approx((m - cm) * kLog2e);
                s0 *= f;
                s1 *= f;
                m = cm;
            }
            const float nm = -m * kLog2e;
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
                s0 += ex2_approx(fmaf(__uint_as_float(r[j]), kLog2e, nm));
                s1 += ex2_approx(fmaf(__uint_as_float(r[j + 1]), kLog2e, nm));
            }
            if ((ycol >> 5) == c && ycol >= 0) {
                const int jj = ycol & 31;
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (j == jj) zyv = __uint_as_float(r[j]);
            }
        }
        if (row < p.T) {
            const size_t o = (size_t)(n0 / BN) * (size_t)p.T + (size_t)row;
            p.part_m[o] = m;
            p.part_s[o] = s0 + s1;
            if (ycol >= 0 && ycol < ncols) p.zy[row] = zyv;
        }
    }
    __device__ void finish() {}
};

// per-tile pairs -> lse, log pi(y), row state.  A CTA covers 32 rows; its 8 warps each take every
// 8th tile (loads are coalesced across the 32 rows), and the partial (max, sum) pairs are combined
// through shared memory in double.
constexpr int kMergeRows = 32;
constexpr int kMergeSlices = 8;

__global__ void __launch_bounds__(kMergeRows * kMergeSlices)
head_merge_kernel(int64_t T, int vocab, int n_tiles, const float* __restrict__ part_m,
                  const float* __restrict__ part_s, const float* __restrict__ zy,
                  const int32_t* __restrict__ targets, const uint8_t* __restrict__ mask, Workspace ws) {
    __shared__ float sh_m[kMergeSlices][kMergeRows];
    __shared__ double sh_s[kMergeSlices][kMergeRows];
    const int lane = threadIdx.x & 31, slice = threadIdx.x >> 5;
    const int64_t r = (int64_t)blockIdx.x * kMergeRows + lane;
    float M = -INFINITY;
    double S = 0.0;
    if (r < T) {
        for (int j = slice; j < n_tiles; j += kMergeSlices) M = fmaxf(M, part_m[(size_t)j * T + r]);
        for (int j = slice; j < n_tiles; j += kMergeSlices) {
            const size_t o = (size_t)j * T + r;
            S += (double)part_s[o] * exp((double)part_m[o] - (double)M);
        }
    }
    sh_m[slice][lane] = M;
    sh_s[slice][lane] = S;
    __syncthreads();
    if (slice != 0 || r >= T) return;
    const bool on = mask ? (mask[r] != 0) : true;
    const int32_t y = targets[r];
    if (!on || y < 0 || y >= vocab) {
        ws.row_state[r] = on ? ROW_BAD_TOKEN : ROW_MASKED;
        ws.lse[r] = 0.0;
        ws.token_logp[r] = 0.0;
        ws.row_max[r] = 0.f;
        return;
    }
    float Mr = sh_m[0][lane];
    for (int k = 1; k < kMergeSlices; ++k) Mr = fmaxf(Mr, sh_m[k][lane]);
    double Sr = 0.0;
    for (int k = 0; k < kMergeSlices; ++k)
        if (sh_s[k][lane] > 0.0) Sr += sh_s[k][lane] * exp((double)sh_m[k][lane] - (double)Mr);
    const double lse = (double)Mr + log(Sr);
    ws.lse[r] = lse;
    ws.token_logp[r] = (double)zy[r] - lse;
    ws.row_max[r] = Mr;
    ws.row_state[r] = ROW_OK;
}

// ---- stores through shared memory and TMA -----------------------------------------------------------

// A warp hands 32 rows x 128 bytes (its 32 accumulator lanes x 64 bf16 or 32 floats) to one tiled
// TMA store.  Two 4 KB buffers alternate; a buffer is rewritten only after the store issued two
// steps earlier has finished reading it.  Stores are clipped at the matrix bounds by the TMA unit.
struct WarpStore {
    uint8_t* stage;
    int lane;
    uint32_t n;  // stores issued
    __device__ WarpStore(uint8_t* s, int l) : stage(s), lane(l), n(0) {}
    __device__ uint8_t* begin() {
        if (n >= 2) {
            if (lane == 0) bulk_wait_read<1>();
            __syncwarp();
        }
        return stage + (n & 1u) * 4096u;
    }
    __device__ void commit(const CUtensorMap* map, uint8_t* buf, int x, int y, bool add = false) {
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
            if (add) tma_reduce_add_2d(map, buf, x, y);
            else tma_store_2d(map, buf, x, y);
            bulk_commit();
        }
        ++n;
    }
    __device__ void finish() {
        if (lane == 0) bulk_wait_all<0>();
        __syncwarp();
    }
};

// ---- forward epilogue with stored logits: bf16(z) to memory, statistics of the rounded values ----------

struct FwdStatsStore {
    struct Params {
        CUtensorMap map;  // z [T, V] bf16, box 64 x 32
        float* part_m;
        float* part_s;
        float* zy;
        const int32_t* targets;
        int T, V;
    };
    const Params& p;
    const int quarter, lane;
    WarpStore st;
    __device__ FwdStatsStore(const Params& p_, uint8_t* stage, int q, int l) : p(p_), quarter(q), lane(l), st(stage, l) {}

    __device__ void tile(int m0, int n0, uint32_t taddr) {
        const int row = m0 + quarter * 32 + lane;
        const int ncols = min(BN, p.V - n0);
        const int ycol = (row < p.T) ? (p.targets[row] - n0) : -1;
        float m = -INFINITY, s0 = 0.f, s1 = 0.f, zyv = 0.f;
#pragma unroll 1
        for (int q = 0; q * 64 < ncols; ++q) {
            uint8_t* buf = st.begin();
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int cc = q * 2 + half;
                uint32_t r[32];
                tmem_ld32(taddr + cc * 32, r);
                tmem_ld_wait();
                uint32_t o[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) o[j] = pack_bf16x2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    *reinterpret_cast<uint4*>(buf + swz128(lane, half * 4 + k)) =
                        make_uint4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
                if (cc * 32 >= ncols) continue;  // this half lies beyond the vocabulary
                // what later steps will read back is the rounded value: the statistics are taken of it
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    r[2 * j] = (cc * 32 + 2 * j < ncols) ? (o[j] << 16) : 0xff800000u;
                    r[2 * j + 1] = (cc * 32 + 2 * j + 1 < ncols) ? (o[j] & 0xffff0000u) : 0xff800000u;
                }
                float cm = __uint_as_float(r[0]);
#pragma unroll
                for (int j = 1; j < 32; ++j) cm = fmaxf(cm, __uint_as_float(r[j]));
                if (cm > m) {
                    const float f = ex2_approx((m - cm) * kLog2e);
                    s0 *= f;
                    s1 *= f;
                    m = cm;
                }
                const float nm = -m * kLog2e;
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    s0 += ex2_approx(fmaf(__uint_as_float(r[j]), kLog2e, nm));
                    s1 += ex2_approx(fmaf(__uint_as_float(r[j + 1]), kLog2e, nm));
                }
                if ((ycol >> 5) == cc && ycol >= 0) {
                    const int jj = ycol & 31;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j == jj) zyv = __uint_as_float(r[j]);
                }
            }
            st.commit(&p.map, buf, n0 + q * 64, m0 + quarter * 32);
        }
        if (row < p.T) {
            const size_t o = (size_t)(n0 / BN) * (size_t)p.T + (size_t)row;
            p.part_m[o] = m;
            p.part_s[o] = s0 + s1;
            if (ycol >= 0 && ycol < ncols) p.zy[row] = zyv;
        }
    }
    __device__ void finish() { st.finish(); }
};

// ---- backward epilogue 1: dz in bf16 -------------------------------------------------------------------

struct DzStore {
    struct Params {
        CUtensorMap map;  // dz [T, V] bf16, box 64 x 32
        const double* lse;
        const double* coef;
        const double* coef_log2;
        const uint8_t* row_state;
        const int32_t* targets;
        int T, V, seq_len;  // T: rows of this chunk
        int row0;           // global index of the chunk's first row (per-row arrays are global)
    };
    const Params& p;
    const int quarter, lane;
    WarpStore st;
    __device__ DzStore(const Params& p_, uint8_t* stage, int q, int l) : p(p_), quarter(q), lane(l), st(stage, l) {}

    __device__ void tile(int m0, int n0, uint32_t taddr) {
        const int row_in_chunk = m0 + quarter * 32 + lane;
        const int row = p.row0 + row_in_chunk;
        const int ncols = min(BN, p.V - n0);
        float c = -INFINITY, g = 0.f;  // dead row: 2^-inf = 0 everywhere, nothing subtracted
        uint32_t sign2 = 0;
        int ycol = -1;
        bool live = false;       // the row has a gradient; otherwise exact zeros, whatever z holds
        if (row_in_chunk < p.T && p.row_state[row] == ROW_OK) {
            const int n = row / p.seq_len;
            const double gd = p.coef[n];
            if (gd != 0.0) {
                c = (float)fma(-p.lse[row], kLog2eD, p.coef_log2[n]);
                g = (float)gd;
                sign2 = (gd < 0.0) ? 0x80008000u : 0u;
                ycol = p.targets[row] - n0;
                live = true;
            }
        }
#pragma unroll 1
        for (int q = 0; q * 64 < ncols; ++q) {
            uint8_t* buf = st.begin();
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int cc = q * 2 + half;
                uint32_t r[32];
                tmem_ld32(taddr + cc * 32, r);
                tmem_ld_wait();
                uint32_t o[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float lo = ex2_approx(fmaf(__uint_as_float(r[2 * j]), kLog2e, c));
                    const float hi = ex2_approx(fmaf(__uint_as_float(r[2 * j + 1]), kLog2e, c));
                    o[j] = (live ? pack_bf16x2(lo, hi) : 0u) ^ sign2;
                }
                if (ycol >= 0 && (ycol >> 5) == cc) {  // the sampled token: g (p_y - 1), formed in float
                    const int jj = ycol & 31;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (j == (jj >> 1)) {
                            const float lo = ex2_approx(fmaf(__uint_as_float(r[2 * j]), kLog2e, c));
                            const float hi = ex2_approx(fmaf(__uint_as_float(r[2 * j + 1]), kLog2e, c));
                            float vlo = (g < 0.f) ? -lo : lo, vhi = (g < 0.f) ? -hi : hi;
                            if (jj & 1) vhi -= g; else vlo -= g;
                            o[j] = pack_bf16x2(vlo, vhi);
                        }
                    }
                }
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    *reinterpret_cast<uint4*>(buf + swz128(lane, half * 4 + k)) =
                        make_uint4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
            }
            st.commit(&p.map, buf, n0 + q * 64, m0 + quarter * 32);
        }
    }
    __device__ void finish() { st.finish(); }
};

// ---- backward epilogues 2 and 3: plain stores ------------------------------------------------------------

struct StoreBf16 {  // dh; dW when the caller wants it in bf16
    struct Params {
        CUtensorMap map;  // [M, N] bf16, box 64 x 32
        int N;
        int accumulate;   // add to what is there (dW, second and later row chunks) instead of overwriting
    };
    const Params& p;
    const int quarter, lane;
    WarpStore st;
    __device__ StoreBf16(const Params& p_, uint8_t* stage, int q, int l) : p(p_), quarter(q), lane(l), st(stage, l) {}
    __device__ void tile(int m0, int n0, uint32_t taddr) {
        const int ncols = min(BN, p.N - n0);
#pragma unroll 1
        for (int q = 0; q * 64 < ncols; ++q) {
            uint8_t* buf = st.begin();
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t r[32];
                tmem_ld32(taddr + (q * 2 + half) * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    uint32_t o[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        o[j] = pack_bf16x2(__uint_as_float(r[8 * k + 2 * j]), __uint_as_float(r[8 * k + 2 * j + 1]));
                    *reinterpret_cast<uint4*>(buf + swz128(lane, half * 4 + k)) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
            st.commit(&p.map, buf, n0 + q * 64, m0 + quarter * 32, p.accumulate != 0);
        }
    }
    __device__ void finish() { st.finish(); }
};

struct StoreF32 {  // dW
    struct Params {
        CUtensorMap map;  // [M, N] float, box 32 x 32
        int N;
        int accumulate;  // add to what is there (second and later row chunks) instead of overwriting
    };
    const Params& p;
    const int quarter, lane;
    WarpStore st;
    __device__ StoreF32(const Params& p_, uint8_t* stage, int q, int l) : p(p_), quarter(q), lane(l), st(stage, l) {}
    __device__ void tile(int m0, int n0, uint32_t taddr) {
        const int ncols = min(BN, p.N - n0);
#pragma unroll 1
        for (int c = 0; c * 32 < ncols; ++c) {
            uint8_t* buf = st.begin();
            uint32_t r[32];
            tmem_ld32(taddr + c * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 8; ++k)
                *reinterpret_cast<uint4*>(buf + swz128(lane, k)) =
                    make_uint4(r[4 * k], r[4 * k + 1], r[4 * k + 2], r[4 * k + 3]);
            st.commit(&p.map, buf, n0 + c * 32, m0 + quarter * 32, p.accumulate != 0);
        }
    }
    __device__ void finish() { st.finish(); }
};

__global__ void clear_status_kernel(int* status) { *status = 0; }

// the status word of the scratch -> the statistics block(s), after everything else
__global__ void publish_status_kernel(const int* status, rapid_stats_t* a, rapid_stats_t* b) {
    if (*status != 0) {
        if (a) atomicMax(&a->status, *status);
        if (b) atomicMax(&b->status, *status);
    }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

rapid_status_t check_head_args(const rapid_desc_t* d, int32_t D) {
    if (!d) return RAPID_ERR_INVALID_ARG;
    if (d->n_seq <= 0 || d->n_groups <= 0 || d->seq_len <= 0 || d->vocab <= 0 || D <= 0) return RAPID_ERR_INVALID_ARG;
    if (!(d->eta > 0.0)) return RAPID_ERR_INVALID_ARG;
    if ((d->flags & RAPID_FLAG_NORM_GIVEN) && !(d->norm_z > 0.0 && d->norm_z < INFINITY)) return RAPID_ERR_INVALID_ARG;
    if (d->dtype != RAPID_BF16) return RAPID_ERR_INVALID_ARG;
    if (d->ld < d->vocab) return RAPID_ERR_INVALID_ARG;
    if (d->flags & RAPID_FLAG_ADV_INPUT_IS_WEIGHT) return RAPID_ERR_INVALID_ARG;
    if (d->ld % 8 != 0 || D % 8 != 0) return RAPID_ERR_ALIGNMENT;  // 16-byte row pitches for TMA
    return RAPID_OK;
}

}  // namespace

}  // namespace rapid

using namespace rapid;
using namespace rapid::umma;

extern "C" rapid_status_t rapid_fused_head_workspace_bytes(const rapid_desc_t* desc, int32_t hidden_dim,
                                                           size_t* bytes) {
    if (!bytes) return RAPID_ERR_INVALID_ARG;
    rapid_status_t s = check_head_args(desc, hidden_dim);
    if (s != RAPID_OK) return s;
    const size_t base = align_up(carve_workspace(*desc, nullptr, nullptr), 1024);
    *bytes = carve_head(*desc, nullptr, base, nullptr);
    return RAPID_OK;
}

extern "C" rapid_status_t rapid_pg_loss_fused_head(
    const rapid_desc_t* desc, int32_t hidden_dim, const void* hidden, const void* w_vocab,
    const int32_t* targets, const uint8_t* mask, const float* behav_logp, const float* rewards,
    const int32_t* group_offsets, float* loss, void* dhidden, void* dW, float* token_logp, float* adv,
    rapid_stats_t* stats, void* workspace, size_t workspace_bytes, void* stream) {
    rapid_status_t s = check_head_args(desc, hidden_dim);
    if (s != RAPID_OK) return s;
    if (!hidden || !w_vocab || !targets || !behav_logp || !rewards || !group_offsets || !loss || !dhidden || !dW)
        return RAPID_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(w_vocab) || !aligned16(dhidden) || !aligned16(dW)) return RAPID_ERR_ALIGNMENT;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) % 1024) != 0) return RAPID_ERR_WORKSPACE;
    Workspace ws;
    HeadScratch hs;
    const size_t base = align_up(carve_workspace(*desc, workspace, &ws), 1024);
    const size_t need = carve_head(*desc, workspace, base, &hs);
    if (workspace_bytes < need) return RAPID_ERR_WORKSPACE;

    int dev = 0, major = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RAPID_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return RAPID_ERR_CUDA;
    if (major != 10) return RAPID_ERR_UNSUPPORTED;

    const int64_t T = (int64_t)desc->n_seq * desc->seq_len;
    const int V = desc->vocab, D = hidden_dim;
    const int64_t ld = desc->ld;
    if (T > 0x7fffffff) return RAPID_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // tensor maps (host structs, passed to the kernels by value)
    CUtensorMap h_k, w_mn, w_k;
    bool ok = make_map_bf16(&h_k, hidden, T, D, D, BK, BM)        // A of forward: rows x K
              && make_map_bf16(&w_mn, w_vocab, D, V, ld, 64, BK)  // B of forward and recompute: K x N
              && make_map_bf16(&w_k, w_vocab, D, V, ld, BK, BN);  // B of dh: N(=D) x K(=V)
    if (!ok) return RAPID_ERR_CUDA;

    const int nV = (V + BN - 1) / BN;
    clear_status_kernel<<<1, 1, 0, st>>>(hs.status);
    // one CTA per 128 x 256 tile, or a pair of CTAs per 256 x 256 tile
    // Which contractions run on pairs of CTAs (one 256 x 256 tile per two SMs) rather than one CTA per
    // 128 x 256 tile: bit 0 forward, 1 recompute, 2 dhidden, 3 dW.  Unless a flag says otherwise the two
    // whose K loop is the hidden size (short, with a heavy epilogue) go to pairs and the two with long K
    // loops stay on single CTAs: measured best on the 16384 x 1536 x 151936 configuration at the power cap
    // (23.45 ms against 24.08 all single and 24.9 all pairs on the same box; pairs need less operand traffic
    // per flop but draw more power, and the long step settles at a lower clock).
    const uint32_t pair_mask = (desc->flags & RAPID_FLAG_HEAD_CTA_PAIRS) ? 15u
                               : (desc->flags & RAPID_FLAG_HEAD_SINGLE_CTA) ? 0u : 3u;
    const bool pairs = (pair_mask & 4u) != 0;
    const bool dw_bf16 = (desc->flags & RAPID_FLAG_HEAD_DW_BF16) != 0;  // dW is [D, ld] bf16 instead of float
    CUtensorMap w_k_half;  // B of dh for a CTA of a pair: 128 of the tile's 256 rows of W^T per box
    if (pairs && !make_map_bf16(&w_k_half, w_vocab, D, V, ld, BK, BN / 2)) return RAPID_ERR_CUDA;

    // forward
    const bool store_z = (desc->flags & RAPID_FLAG_HEAD_STORE_LOGITS) != 0;
    {
        Shape fwd{(int)((T + BM - 1) / BM), nV, (D + BK - 1) / BK, M_FASTEST};
        if (store_z) {
            FwdStatsStore::Params fp;
            if (!make_map_bf16(&fp.map, hs.dz, T, V, hs.ldz, 64, 32)) return RAPID_ERR_CUDA;
            fp.part_m = hs.part_m;
            fp.part_s = hs.part_s;
            fp.zy = hs.zy;
            fp.targets = targets;
            fp.T = (int)T;
            fp.V = V;
            if (((pair_mask & 1u) ? launch_gemm_pair<FwdStatsStore, false, true>(h_k, w_mn, fwd, sms, hs.status, fp, st)
                       : launch_gemm<FwdStatsStore, false, true>(h_k, w_mn, fwd, sms, hs.status, fp, st)) != cudaSuccess)
                return RAPID_ERR_CUDA;
        } else {
            FwdStats::Params fp{hs.part_m, hs.part_s, hs.zy, targets, (int)T, V};
            if (((pair_mask & 1u) ? launch_gemm_pair<FwdStats, false, true>(h_k, w_mn, fwd, sms, hs.status, fp, st)
                       : launch_gemm<FwdStats, false, true>(h_k, w_mn, fwd, sms, hs.status, fp, st)) != cudaSuccess)
                return RAPID_ERR_CUDA;
        }
    }
    head_merge_kernel<<<(unsigned)((T + kMergeRows - 1) / kMergeRows), kMergeRows * kMergeSlices, 0, st>>>(
        T, V, hs.n_tiles, hs.part_m, hs.part_s, hs.zy, targets, mask, ws);
    if (cudaGetLastError() != cudaSuccess) return RAPID_ERR_CUDA;
    if (launch_seq_reduce(*desc, behav_logp, token_logp, ws, st) != cudaSuccess) return RAPID_ERR_CUDA;
    if (launch_finalize(*desc, rewards, group_offsets, loss, adv, stats, ws, st) != cudaSuccess) return RAPID_ERR_CUDA;

    // with stored logits: dlogits in place, by the second pass of the logits-in path
    if (store_z) {
        rapid_desc_t dz_desc = *desc;
        dz_desc.ld = hs.ldz;
        if (launch_dlogits(dz_desc, hs.dz, hs.dz, 0, T, targets, stats, ws, sms, st) != cudaSuccess) return RAPID_ERR_CUDA;
    }

    // backward, a chunk of rows at a time: dz (recompute), then dh for those rows and the chunk's
    // contribution to dW (the first chunk overwrites dW, later ones add to it, in stream order)
    for (int64_t r0 = 0; r0 < T; r0 += kHeadChunkRows) {
        const int64_t R = (T - r0 < kHeadChunkRows) ? T - r0 : kHeadChunkRows;
        const uint16_t* h_c = static_cast<const uint16_t*>(hidden) + (size_t)r0 * D;
        uint16_t* dh_c = static_cast<uint16_t*>(dhidden) + (size_t)r0 * D;
        uint16_t* dz_c = hs.dz + (store_z ? (size_t)r0 * (size_t)hs.ldz : 0);  // the chunk's rows of dlogits
        CUtensorMap hc_k, hc_mn, dz_k, dz_mn;
        DzStore::Params dzp;
        StoreBf16::Params dhp;
        StoreF32::Params dwp;
        StoreBf16::Params dwp16;
        ok = make_map_bf16(&hc_k, h_c, R, D, D, BK, BM)                // A of recompute: rows x K
             && make_map_bf16(&hc_mn, h_c, R, D, D, 64, BK)            // A of dW: K(=rows) x M(=D)
             && make_map_bf16(&dz_k, dz_c, R, V, hs.ldz, BK, BM)      // A of dh: rows x K(=V)
             && make_map_bf16(&dz_mn, dz_c, R, V, hs.ldz, 64, BK)     // B of dW: K(=rows) x N(=V)
             && make_map_bf16(&dzp.map, dz_c, R, V, hs.ldz, 64, 32)   // stores
             && make_map_bf16(&dhp.map, dh_c, R, D, D, 64, 32)
             && (dw_bf16 ? make_map_bf16(&dwp16.map, dW, D, V, ld, 64, 32) : make_map_f32(&dwp.map, dW, D, V, ld, 32, 32));
        if (!ok) return RAPID_ERR_CUDA;
        const int mR = (int)((R + BM - 1) / BM);

        dzp.lse = ws.lse;
        dzp.coef = ws.coef;
        dzp.coef_log2 = ws.coef_log2;
        dzp.row_state = ws.row_state;
        dzp.targets = targets;
        dzp.T = (int)R;
        dzp.V = V;
        dzp.seq_len = desc->seq_len;
        dzp.row0 = (int)r0;
        Shape sdz{mR, nV, (D + BK - 1) / BK, M_FASTEST};
        if (!store_z && ((pair_mask & 2u) ? launch_gemm_pair<DzStore, false, true>(hc_k, w_mn, sdz, sms, hs.status, dzp, st)
                               : launch_gemm<DzStore, false, true>(hc_k, w_mn, sdz, sms, hs.status, dzp, st)) != cudaSuccess)
            return RAPID_ERR_CUDA;

        dhp.N = D;
        dhp.accumulate = 0;
        Shape sdh{mR, (D + BN - 1) / BN, (V + BK - 1) / BK, N_FASTEST};
        if (((pair_mask & 4u) ? launch_gemm_pair<StoreBf16, false, false>(dz_k, w_k_half, sdh, sms, hs.status, dhp, st)
                   : launch_gemm<StoreBf16, false, false>(dz_k, w_k, sdh, sms, hs.status, dhp, st)) != cudaSuccess)
            return RAPID_ERR_CUDA;

        dwp.N = dwp16.N = V;
        dwp.accumulate = dwp16.accumulate = (r0 > 0) ? 1 : 0;
        Shape sdw{(D + BM - 1) / BM, nV, (int)((R + BK - 1) / BK), M_FASTEST};
        cudaError_t ew;
        if (dw_bf16)
            ew = (pair_mask & 8u) ? launch_gemm_pair<StoreBf16, true, true>(hc_mn, dz_mn, sdw, sms, hs.status, dwp16, st)
                                  : launch_gemm<StoreBf16, true, true>(hc_mn, dz_mn, sdw, sms, hs.status, dwp16, st);
        else
            ew = (pair_mask & 8u) ? launch_gemm_pair<StoreF32, true, true>(hc_mn, dz_mn, sdw, sms, hs.status, dwp, st)
                                  : launch_gemm<StoreF32, true, true>(hc_mn, dz_mn, sdw, sms, hs.status, dwp, st);
        if (ew != cudaSuccess) return RAPID_ERR_CUDA;
    }

    publish_status_kernel<<<1, 1, 0, st>>>(hs.status, stats, ws.stats);
    return cudaGetLastError() == cudaSuccess ? RAPID_OK : RAPID_ERR_CUDA;
}
