// rapid_pg_loss_fwd_bwd_noalloc: the one-call path for callers that cannot provide a workspace
// because they cannot allocate device memory.  The scratch lives in a fixed array inside this
// library's device image; see include/rapid_pg.h for the contract.
//
// The array's name is usable directly only in device code.  In host code the name is a host-side
// handle, NOT a device address: handing it to a kernel would make the kernel fault (or, on
// systems where the GPU can reach host memory, quietly scribble over the wrong bytes).  The host
// therefore asks the runtime for the array's device address, with the caller's device current, and
// passes that pointer on.  The address is asked for on EVERY call and never remembered: after the
// first call on a device the query is a host-side table look-up, and an address remembered across a
// cudaDeviceReset, or used under another context on the same device ordinal, would be stale.
#include "rapid_common.cuh"

namespace {

// One array per device that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[RAPID_NOALLOC_SCRATCH_BYTES];

// Device address of the scratch array on the CURRENT device.
rapid_status_t scratch_for_current_device(void** out) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
        (void)cudaGetLastError();  // leave no sticky-looking error behind for the caller
        return RAPID_ERR_CUDA;
    }
    *out = ptr;
    return RAPID_OK;
}

}  // namespace

extern "C" rapid_status_t rapid_pg_loss_fwd_bwd_noalloc(
    const rapid_desc_t* desc, const void* logits, const int32_t* targets, const uint8_t* mask,
    const float* behav_logp, const float* rewards, const int32_t* group_offsets, void* dlogits,
    float* loss, float* token_logp, float* adv, rapid_stats_t* stats, void* stream) {
    // Size first, on the host alone: a problem that does not fit is refused before the device is
    // touched.  rapid_workspace_bytes also rejects a malformed descriptor.
    size_t need = 0;
    rapid_status_t s = rapid_workspace_bytes(desc, &need);
    if (s != RAPID_OK) return s;
    if (need > (size_t)RAPID_NOALLOC_SCRATCH_BYTES) return RAPID_ERR_UNSUPPORTED;
    void* scratch = nullptr;
    if ((s = scratch_for_current_device(&scratch)) != RAPID_OK) return s;
    // Nothing in the scratch has to start at zero: every word a later kernel reads (per-row state,
    // per-generation sums, the statistics block) is rewritten earlier in the same call, so the
    // previous call's leftovers are never seen.
    return rapid_pg_loss_fwd_bwd(desc, logits, targets, mask, behav_logp, rewards, group_offsets,
                                 dlogits, loss, token_logp, adv, stats, scratch,
                                 (size_t)RAPID_NOALLOC_SCRATCH_BYTES, stream);
}
