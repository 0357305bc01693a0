// The C ABI of librapid_pg: host-side argument checks, workspace carving and kernel launches.
// Nothing here allocates, synchronises or keeps state (the one call that works in a library-owned
// array is in noalloc.cu); see include/rapid_pg.h for the contract.
#include <math.h>

#include "rapid_common.cuh"

using namespace rapid;

namespace {

constexpr int32_t kVersion = 100;  // 0.1.0

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t elem_size(int32_t dtype) { return dtype == RAPID_BF16 ? 2 : 4; }

rapid_status_t check_desc_basic(const rapid_desc_t* d) {
    if (!d) return RAPID_ERR_INVALID_ARG;
    if (d->n_seq <= 0 || d->n_groups <= 0) return RAPID_ERR_INVALID_ARG;
    if (!(d->eta > 0.0)) return RAPID_ERR_INVALID_ARG;  // also rejects NaN
    if ((d->flags & RAPID_FLAG_NORM_GIVEN) && !(d->norm_z > 0.0 && d->norm_z < INFINITY)) return RAPID_ERR_INVALID_ARG;
    return RAPID_OK;
}

rapid_status_t check_desc_full(const rapid_desc_t* d) {
    rapid_status_t s = check_desc_basic(d);
    if (s != RAPID_OK) return s;
    if (d->seq_len <= 0 || d->vocab <= 0) return RAPID_ERR_INVALID_ARG;
    if (d->dtype != RAPID_F32 && d->dtype != RAPID_BF16) return RAPID_ERR_INVALID_ARG;
    if (d->ld < d->vocab) return RAPID_ERR_INVALID_ARG;
    if (((size_t)d->ld * elem_size(d->dtype)) % 16 != 0) return RAPID_ERR_ALIGNMENT;
    if (d->flags & RAPID_FLAG_ADV_INPUT_IS_WEIGHT) return RAPID_ERR_INVALID_ARG;
    return RAPID_OK;
}

rapid_status_t check_workspace(const rapid_desc_t* d, const void* ws, size_t bytes, Workspace* out) {
    if (!ws || !aligned(ws, 256)) return RAPID_ERR_WORKSPACE;
    const size_t need = carve_workspace(*d, const_cast<void*>(ws), out);
    if (bytes < need) return RAPID_ERR_WORKSPACE;
    return RAPID_OK;
}

// sm_100 only.  Returns the SM count of the current device through *sm_count.
rapid_status_t check_device(int* sm_count) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RAPID_ERR_CUDA;
    int major = 0, minor = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return RAPID_ERR_CUDA;
    if (major != 10) return RAPID_ERR_UNSUPPORTED;
    *sm_count = sms;
    return RAPID_OK;
}

inline rapid_status_t cuda_status(cudaError_t e) { return e == cudaSuccess ? RAPID_OK : RAPID_ERR_CUDA; }

}  // namespace

extern "C" {

const char* rapid_status_string(rapid_status_t status) {
    switch (status) {
        case RAPID_OK: return "RAPID_OK";
        case RAPID_ERR_INVALID_ARG: return "RAPID_ERR_INVALID_ARG";
        case RAPID_ERR_ALIGNMENT: return "RAPID_ERR_ALIGNMENT";
        case RAPID_ERR_UNSUPPORTED: return "RAPID_ERR_UNSUPPORTED";
        case RAPID_ERR_WORKSPACE: return "RAPID_ERR_WORKSPACE";
        case RAPID_ERR_CUDA: return "RAPID_ERR_CUDA";
        case RAPID_ERR_TIMEOUT: return "RAPID_ERR_TIMEOUT";
    }
    return "RAPID_ERR_UNKNOWN";
}

int32_t rapid_version(void) { return kVersion; }

rapid_status_t rapid_workspace_bytes(const rapid_desc_t* desc, size_t* bytes) {
    if (!bytes) return RAPID_ERR_INVALID_ARG;
    rapid_status_t s = check_desc_full(desc);
    if (s != RAPID_OK) return s;
    *bytes = carve_workspace(*desc, nullptr, nullptr);
    return RAPID_OK;
}

rapid_status_t rapid_group_advantage(const rapid_desc_t* desc, const float* rewards,
                                     const double* seq_log_ratio, const int32_t* group_offsets,
                                     float* adv, double* clipped_w, rapid_stats_t* stats,
                                     void* stream) {
    rapid_status_t s = check_desc_basic(desc);
    if (s != RAPID_OK) return s;
    if (!rewards || !group_offsets || !adv) return RAPID_ERR_INVALID_ARG;
    int sms = 0;
    if ((s = check_device(&sms)) != RAPID_OK) return s;
    return cuda_status(launch_group_advantage(*desc, rewards, seq_log_ratio, group_offsets, adv,
                                              clipped_w, stats, static_cast<cudaStream_t>(stream)));
}

rapid_status_t rapid_pg_stats_chunk(const rapid_desc_t* desc, const void* logits_chunk,
                                    int64_t row0, int64_t n_rows, const int32_t* targets,
                                    const uint8_t* mask, void* workspace, size_t workspace_bytes,
                                    void* stream) {
    rapid_status_t s = check_desc_full(desc);
    if (s != RAPID_OK) return s;
    const int64_t T = (int64_t)desc->n_seq * desc->seq_len;
    if (!logits_chunk || !targets) return RAPID_ERR_INVALID_ARG;
    if (row0 < 0 || n_rows < 0 || row0 + n_rows > T) return RAPID_ERR_INVALID_ARG;
    if (!aligned(logits_chunk, 16)) return RAPID_ERR_ALIGNMENT;
    Workspace ws;
    if ((s = check_workspace(desc, workspace, workspace_bytes, &ws)) != RAPID_OK) return s;
    int sms = 0;
    if ((s = check_device(&sms)) != RAPID_OK) return s;
    return cuda_status(launch_row_stats(*desc, logits_chunk, row0, n_rows, targets, mask, ws, sms,
                                        static_cast<cudaStream_t>(stream)));
}

rapid_status_t rapid_pg_finalize(const rapid_desc_t* desc, const float* behav_logp,
                                 const float* rewards, const int32_t* group_offsets, float* loss,
                                 float* token_logp, float* adv, rapid_stats_t* stats,
                                 void* workspace, size_t workspace_bytes, void* stream) {
    rapid_status_t s = check_desc_full(desc);
    if (s != RAPID_OK) return s;
    if (!behav_logp || !rewards || !group_offsets || !loss) return RAPID_ERR_INVALID_ARG;
    Workspace ws;
    if ((s = check_workspace(desc, workspace, workspace_bytes, &ws)) != RAPID_OK) return s;
    int sms = 0;
    if ((s = check_device(&sms)) != RAPID_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = launch_seq_reduce(*desc, behav_logp, token_logp, ws, st);
    if (e != cudaSuccess) return RAPID_ERR_CUDA;
    return cuda_status(launch_finalize(*desc, rewards, group_offsets, loss, adv, stats, ws, st));
}

rapid_status_t rapid_pg_dlogits_chunk(const rapid_desc_t* desc, const void* logits_chunk,
                                      void* dlogits_chunk, int64_t row0, int64_t n_rows,
                                      const int32_t* targets, rapid_stats_t* stats,
                                      void* workspace, size_t workspace_bytes, void* stream) {
    rapid_status_t s = check_desc_full(desc);
    if (s != RAPID_OK) return s;
    const int64_t T = (int64_t)desc->n_seq * desc->seq_len;
    if (!logits_chunk || !dlogits_chunk || !targets) return RAPID_ERR_INVALID_ARG;
    if (row0 < 0 || n_rows < 0 || row0 + n_rows > T) return RAPID_ERR_INVALID_ARG;
    if (!aligned(logits_chunk, 16) || !aligned(dlogits_chunk, 16)) return RAPID_ERR_ALIGNMENT;
    if (logits_chunk != dlogits_chunk) {  // partial overlap is not allowed
        const size_t span = (size_t)n_rows * (size_t)desc->ld * elem_size(desc->dtype);
        const uintptr_t a = reinterpret_cast<uintptr_t>(logits_chunk);
        const uintptr_t b = reinterpret_cast<uintptr_t>(dlogits_chunk);
        if (a < b + span && b < a + span) return RAPID_ERR_INVALID_ARG;
    }
    Workspace ws;
    if ((s = check_workspace(desc, workspace, workspace_bytes, &ws)) != RAPID_OK) return s;
    int sms = 0;
    if ((s = check_device(&sms)) != RAPID_OK) return s;
    return cuda_status(launch_dlogits(*desc, logits_chunk, dlogits_chunk, row0, n_rows, targets, stats,
                                      ws, sms, static_cast<cudaStream_t>(stream)));
}

rapid_status_t rapid_pg_loss_fwd_bwd(const rapid_desc_t* desc, const void* logits,
                                     const int32_t* targets, const uint8_t* mask,
                                     const float* behav_logp, const float* rewards,
                                     const int32_t* group_offsets, void* dlogits, float* loss,
                                     float* token_logp, float* adv, rapid_stats_t* stats,
                                     void* workspace, size_t workspace_bytes, void* stream) {
    rapid_status_t s = check_desc_full(desc);
    if (s != RAPID_OK) return s;
    // check everything before the first launch so that a bad argument enqueues nothing
    if (!logits || !targets || !behav_logp || !rewards || !group_offsets || !dlogits || !loss)
        return RAPID_ERR_INVALID_ARG;
    if (!aligned(logits, 16) || !aligned(dlogits, 16)) return RAPID_ERR_ALIGNMENT;
    const int64_t T = (int64_t)desc->n_seq * desc->seq_len;
    if (logits != dlogits) {
        const size_t span = (size_t)T * (size_t)desc->ld * elem_size(desc->dtype);
        const uintptr_t a = reinterpret_cast<uintptr_t>(logits);
        const uintptr_t b = reinterpret_cast<uintptr_t>(dlogits);
        if (a < b + span && b < a + span) return RAPID_ERR_INVALID_ARG;
    }
    Workspace ws;
    if ((s = check_workspace(desc, workspace, workspace_bytes, &ws)) != RAPID_OK) return s;
    s = rapid_pg_stats_chunk(desc, logits, 0, T, targets, mask, workspace, workspace_bytes, stream);
    if (s != RAPID_OK) return s;
    s = rapid_pg_finalize(desc, behav_logp, rewards, group_offsets, loss, token_logp, adv, stats,
                          workspace, workspace_bytes, stream);
    if (s != RAPID_OK) return s;
    return rapid_pg_dlogits_chunk(desc, logits, dlogits, 0, T, targets, stats, workspace,
                                  workspace_bytes, stream);
}

rapid_status_t rapid_pg_loss_fwd_bwd_hostlogits(const rapid_desc_t* desc, const void* logits_host,
                                                void* logits_staging, const int32_t* targets,
                                                const uint8_t* mask, const float* behav_logp,
                                                const float* rewards, const int32_t* group_offsets,
                                                void* dlogits, float* loss, float* token_logp, float* adv,
                                                rapid_stats_t* stats, void* workspace,
                                                size_t workspace_bytes, void* stream) {
    rapid_status_t s = check_desc_full(desc);
    if (s != RAPID_OK) return s;
    if (!logits_host || !logits_staging || !targets || !behav_logp || !rewards || !group_offsets || !dlogits ||
        !loss)
        return RAPID_ERR_INVALID_ARG;
    if (!aligned(logits_host, 16) || !aligned(logits_staging, 16) || !aligned(dlogits, 16)) return RAPID_ERR_ALIGNMENT;
    const int64_t T = (int64_t)desc->n_seq * desc->seq_len;
    if (logits_staging != dlogits) {
        const size_t span = (size_t)T * (size_t)desc->ld * elem_size(desc->dtype);
        const uintptr_t a = reinterpret_cast<uintptr_t>(logits_staging);
        const uintptr_t b = reinterpret_cast<uintptr_t>(dlogits);
        if (a < b + span && b < a + span) return RAPID_ERR_INVALID_ARG;
    }
    Workspace ws;
    if ((s = check_workspace(desc, workspace, workspace_bytes, &ws)) != RAPID_OK) return s;
    int sms = 0;
    if ((s = check_device(&sms)) != RAPID_OK) return s;
    // The kernel will dereference logits_host: it must be page-locked host memory that the device can
    // address.  Anything else is refused here rather than left to fault on the device.
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, logits_host) != cudaSuccess) {
        (void)cudaGetLastError();
        return RAPID_ERR_INVALID_ARG;
    }
    if (at.type != cudaMemoryTypeHost || !at.devicePointer) return RAPID_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = launch_row_stats(*desc, at.devicePointer, 0, T, targets, mask, ws, sms, st, logits_staging);
    if (e != cudaSuccess) return RAPID_ERR_CUDA;
    s = rapid_pg_finalize(desc, behav_logp, rewards, group_offsets, loss, token_logp, adv, stats, workspace,
                          workspace_bytes, stream);
    if (s != RAPID_OK) return s;
    return rapid_pg_dlogits_chunk(desc, logits_staging, dlogits, 0, T, targets, stats, workspace,
                                  workspace_bytes, stream);
}

rapid_status_t rapid_pg_loss_onpolicy_fwd_bwd(const rapid_desc_t* desc, const void* logits,
                                              const int32_t* targets, const uint8_t* mask,
                                              const float* rewards, const int32_t* group_offsets,
                                              void* dlogits, float* loss, float* token_logp, float* adv,
                                              rapid_stats_t* stats, void* workspace,
                                              size_t workspace_bytes, void* stream) {
    rapid_status_t s = check_desc_full(desc);
    if (s != RAPID_OK) return s;
    if (!logits || !targets || !rewards || !group_offsets || !dlogits || !loss) return RAPID_ERR_INVALID_ARG;
    if (!aligned(logits, 16) || !aligned(dlogits, 16)) return RAPID_ERR_ALIGNMENT;
    const int64_t T = (int64_t)desc->n_seq * desc->seq_len;
    if (logits != dlogits) {
        const size_t span = (size_t)T * (size_t)desc->ld * elem_size(desc->dtype);
        const uintptr_t a = reinterpret_cast<uintptr_t>(logits);
        const uintptr_t b = reinterpret_cast<uintptr_t>(dlogits);
        if (a < b + span && b < a + span) return RAPID_ERR_INVALID_ARG;
    }
    Workspace ws;
    if ((s = check_workspace(desc, workspace, workspace_bytes, &ws)) != RAPID_OK) return s;
    int sms = 0;
    if ((s = check_device(&sms)) != RAPID_OK) return s;
    return cuda_status(launch_onpolicy(*desc, logits, dlogits, targets, mask, rewards, group_offsets, loss,
                                       token_logp, adv, stats, ws, sms, static_cast<cudaStream_t>(stream)));
}

}  // extern "C"
