/*
 * rapid_pg.h -- C ABI of librapid_pg: the importance-weighted group-advantage policy-gradient
 * loss of RAPID (arXiv 2510.03515) and its gradient w.r.t. the logits, as CUDA kernels for
 * NVIDIA B200 (sm_100a).
 *
 * What one call computes (the two "Compute ..." lines of Algorithm 1, procedure IW-GRPG, for one
 * mini-batch Z_h of N generations):
 *
 *   log pi_theta(y_t|.) = z[r, y_r] - logsumexp_v z[r, v]                  softmax policy, Sec. 3.1
 *   s_n = sum_t m_r (log pi_theta(y_t) - log mu(y_t)),  w_n = exp(s_n)    generation-level weight,
 *                                                                          Sec. 4.3 ("Importance-
 *                                                                          weight clipping")
 *   c_n = min(w_n, eta)                                                    Eq. 5 (cap; eta = 2.0
 *                                                                          in the paper's table of
 *                                                                          hyper-parameters)
 *   A_n = R_n - (1/N_k) sum_{n' in group k} c_n' R_n'                      Eq. 5 (Eq. 2 when every
 *                                                                          c is 1, Eq. 4 when
 *                                                                          eta = +inf)
 *   g_n = c_n A_n / N,   loss = - sum_n g_n sum_t m_r log pi_theta(y_t)    Eq. 3, with
 *                                                                          grad pi / mu = w grad log pi
 *                                                                          and w, A held constant
 *   dlogits[r, v] = g_n m_r (softmax(z[r, .])_v - 1[v == y_r])            d loss / d logits
 *
 * Row r = n * seq_len + t of the padded token grid belongs to generation n.  `loss` is minus the
 * paper's objective estimate (the paper takes ascent steps; this library returns the quantity
 * to minimise), so dlogits = -(w A (onehot - softmax)) / N.
 *
 * Conventions, unless a parameter says otherwise:
 *   - `desc`, `bytes` and other plain scalars are HOST memory; every array pointer is a DEVICE
 *     pointer owned by the caller and valid on the current device.  The library allocates
 *     nothing, frees nothing and keeps no state between calls: everything a call needs beyond its
 *     arguments lives in the caller's workspace.  (One exception, stated at its declaration:
 *     rapid_pg_loss_fwd_bwd_noalloc works in a fixed device array that all its calls share.)
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the default stream)
 *     and the call returns without synchronising.  Outputs are valid once the stream reaches
 *     the end of the enqueued work.
 *   - The return value reports what the host can see (NULL pointers, sizes, alignment, launch
 *     errors).  Problems only the device can see never trap: a sampled token id outside
 *     [0, vocab) makes its row count as masked and is counted in rapid_stats_t.n_bad_token; an
 *     invalid group_offsets array sets rapid_stats_t.status, zeroes every coefficient (so
 *     dlogits is all zero) and makes loss NaN.
 *   - Logits must not be +inf or NaN (results unspecified, but memory-safe).  -inf, or the
 *     dtype's lowest finite value, marks a masked part of the vocabulary and is accepted under the
 *     condition stated at rapid_pg_loss_fwd_bwd.
 *   - Only sm_100 devices are supported: other devices get RAPID_ERR_UNSUPPORTED.
 */
#ifndef RAPID_PG_H
#define RAPID_PG_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RAPID_OK = 0,
    RAPID_ERR_INVALID_ARG = 1, /* NULL where an array is required, non-positive size, ld < vocab  */
    RAPID_ERR_ALIGNMENT = 2,   /* a logits base or row pitch that is not a multiple of 16 bytes   */
    RAPID_ERR_UNSUPPORTED = 3, /* wrong device architecture, or a size beyond a stated limit      */
    RAPID_ERR_WORKSPACE = 4,   /* workspace NULL, misaligned (256 B) or smaller than required     */
    RAPID_ERR_CUDA = 5,        /* a CUDA runtime call or kernel launch failed                     */
    RAPID_ERR_TIMEOUT = 6      /* a bounded device-side wait gave up (reported in stats.status)   */
} rapid_status_t;

typedef enum { RAPID_F32 = 0, RAPID_BF16 = 1 } rapid_dtype_t;

enum {
    /* Eq. 3 exactly as printed: the outer weight is w_n, not the clipped c_n.  Default (flag
     * clear) clips both, which is what keeps generation-level weights from blowing up.          */
    RAPID_FLAG_OUTER_UNCLIPPED = 1u,
    /* Normalise by the number of unmasked tokens instead of the number of generations N.        */
    RAPID_FLAG_NORM_TOKENS = 2u,
    /* rapid_group_advantage only: seq_log_ratio holds w_n itself, not s_n = log w_n.            */
    RAPID_FLAG_ADV_INPUT_IS_WEIGHT = 4u,
    /* Baseline over the other members of the group, divided by N_k - 1 (the unbiased variant
     * shown after Eq. 4, which the paper states but does not use).                              */
    RAPID_FLAG_LEAVE_ONE_OUT = 8u,
    /* With LEAVE_ONE_OUT: divide by N_k, as that display is printed.                            */
    RAPID_FLAG_LOO_LITERAL_DIVISOR = 16u,
    /* The normaliser Z of Eq. 3 is desc->norm_z instead of being counted from this call's own    */
    /* generations (or tokens).  For a mini-batch whose prompt groups are spread over several     */
    /* GPUs: every rank passes the global N (or the global token count), so that the per-rank     */
    /* losses and gradients simply add up to those of the whole mini-batch.                       */
    RAPID_FLAG_NORM_GIVEN = 32u,
    /* rapid_pg_loss_fused_head only: the forward contraction also writes its logits, rounded to   */
    /* bf16, into the workspace, and the backward part turns them into dlogits in place instead of */
    /* forming them a second time on the tensor cores: three GEMM-sized contractions instead of    */
    /* four, for one more write and read of [T, vocab] bf16.  The row statistics are then those of */
    /* the rounded logits, i.e. the results are those of rapid_pg_loss_fwd_bwd on bf16(h W).       */
    RAPID_FLAG_HEAD_STORE_LOGITS = 64u,
    /* rapid_pg_loss_fused_head only.  Its contractions run either on one CTA per 128 x 256 tile or  */
    /* on PAIRS of CTAs (two SMs share one 256 x 256 tile, each holding half of either operand;      */
    /* tcgen05 cta_group::2; every pair is a thread-block cluster on this GPU alone): same results   */
    /* to rounding order, a third less operand traffic into shared memory per flop, more power.  By  */
    /* default the forward and the recompute contraction (K = hidden size) run on pairs and the two  */
    /* long-K ones (dhidden, dW) on single CTAs, the mix measured fastest; these two flags force     */
    /* all four one way (CTA_PAIRS wins if both are given).                                          */
    RAPID_FLAG_HEAD_CTA_PAIRS = 128u,
    RAPID_FLAG_HEAD_SINGLE_CTA = 256u,
    /* rapid_pg_loss_fused_head only: dW is written as bf16 ([D, ld] bf16, same pitch rule as w_vocab) */
    /* instead of float: half the bytes, for a weight gradient that a bf16 optimizer state consumes.  */
    /* The float accumulator is rounded once per backward chunk of 16384 rows; with more rows than    */
    /* that the chunks' contributions are added in bf16, one rounding per chunk.                      */
    RAPID_FLAG_HEAD_DW_BF16 = 512u
};

/* Problem descriptor (host memory, plain data, 48 bytes). */
typedef struct rapid_desc {
    int32_t n_seq;    /* N: generations in the mini-batch (N_step in the paper)                   */
    int32_t seq_len;  /* L: padded response length; rows T = N * L                                */
    int32_t vocab;    /* V                                                                        */
    int32_t n_groups; /* K: prompts; group k is the generation range [offsets[k], offsets[k+1])  */
    int64_t ld;       /* row pitch of logits / dlogits in ELEMENTS, >= vocab, pitch bytes % 16 == 0 */
    int32_t dtype;    /* rapid_dtype_t of logits and dlogits                                      */
    uint32_t flags;   /* RAPID_FLAG_* bits                                                        */
    double eta;       /* importance-weight cap of Eq. 5; +inf gives Eq. 4; must be > 0            */
    double norm_z;    /* Z of Eq. 3 when RAPID_FLAG_NORM_GIVEN is set (> 0, finite); else ignored  */
} rapid_desc_t;

/* Side statistics (DEVICE memory, written by the finalize step, 48 bytes). */
typedef struct rapid_stats {
    int64_t n_tokens;       /* tokens that count: mask set and target id valid                    */
    int32_t n_clipped;      /* generations with w_n > eta (strictly)                              */
    int32_t n_bad_token;    /* rows with mask set but target id outside [0, vocab)                */
    int32_t n_empty_group;  /* groups with N_k = 0 (skipped)                                      */
    int32_t status;         /* rapid_status_t seen by the device: RAPID_OK, or                    */
                            /* RAPID_ERR_INVALID_ARG when group_offsets is not a monotone cover   */
                            /* of [0, N)                                                          */
    double mean_log_cw;     /* (1/N) sum_n log c_n: the staleness statistic of Sec. 4.3 / Table 3 */
    double mean_abs_log_cw; /* (1/N) sum_n |log c_n|                                              */
    double loss;            /* the loss in double                                                 */
} rapid_stats_t;

/*
 * Self-test of the time-out path (the paper has no counterpart: this is a property of the
 * implementation).  The pipelined kernels wait on shared-memory barriers for their bulk copies;
 * every such wait is bounded and, when its limit passes, raises RAPID_ERR_TIMEOUT in the statistics
 * block instead of spinning or trapping.  This call runs that very wait routine in a one-warp kernel
 * on a barrier that nothing arrives at, with a limit of `limit_ns` nanoseconds (1 .. 1e9; more
 * returns RAPID_ERR_UNSUPPORTED, 0 or a NULL `stats` RAPID_ERR_INVALID_ARG).  On completion
 * stats->status == RAPID_ERR_TIMEOUT and stats->n_tokens holds the nanoseconds the wait lasted;
 * the other fields are zero.  `stats` is a DEVICE pointer.  The kernel ends normally and the context
 * stays usable.
 */
rapid_status_t rapid_selftest_bounded_wait(uint64_t limit_ns, rapid_stats_t* stats, void* stream);

/* Human-readable name of a status code (static storage, never NULL). */
const char* rapid_status_string(rapid_status_t status);

/* Library version as major * 10000 + minor * 100 + patch. */
int32_t rapid_version(void);

/*
 * Size of the scratch workspace the logits-in calls need for `desc` (21 bytes per row plus a
 * few per generation).  `bytes` is host memory.  The workspace must be 256-byte aligned device
 * memory; its contents need not be initialised.  Between rapid_pg_stats_chunk, rapid_pg_finalize
 * and rapid_pg_dlogits_chunk it carries the per-row and per-generation state and must not be
 * touched by the caller.  It also holds the counters from which the streaming kernels draw their
 * rows, so calls that use the same workspace must not overlap on the device: put them on one
 * stream, or order them with events (the blocks of the chunked form included).
 */
rapid_status_t rapid_workspace_bytes(const rapid_desc_t* desc, size_t* bytes);

/*
 * Group advantage on its own (Eq. 2 / Eq. 4 / Eq. 5; leave-one-out by flag).
 *   rewards        [N] float, R_n (any finite value)
 *   seq_log_ratio  [N] double, s_n = log w_n (or w_n with RAPID_FLAG_ADV_INPUT_IS_WEIGHT);
 *                  NULL = on-policy, every weight 1 (Eq. 2)
 *   group_offsets  [K+1] int32, offsets[0] = 0, non-decreasing, offsets[K] = N
 *   adv            [N] float out: the double result rounded once to float
 *   clipped_w      [N] double out, c_n; may be NULL
 *   stats          out, may be NULL; only status, n_clipped, n_empty_group, mean_log_cw and
 *                  mean_abs_log_cw are meaningful here (the rest is zero)
 * Uses desc->n_seq, n_groups, eta and flags only.  Sums run in index order in double without
 * fused multiply-add, so the result is bit-identical to the plain definition evaluated the same
 * way whenever the weights are identical.
 */
rapid_status_t rapid_group_advantage(const rapid_desc_t* desc, const float* rewards,
                                     const double* seq_log_ratio, const int32_t* group_offsets,
                                     float* adv, double* clipped_w, rapid_stats_t* stats,
                                     void* stream);

/*
 * The whole path over one mini-batch whose logits are resident: two reads and one write of the
 * logits (a first pass for the row statistics, the per-generation/per-group finalize, and one
 * re-read pass that writes dlogits).
 *   logits        [T, ld] of desc->dtype, row-major; only the first `vocab` entries of a row
 *                 are used.  Base address and ld * sizeof(element) must be multiples of 16.
 *                 Entries may be -inf or the dtype's lowest finite value (a masked part of the
 *                 vocabulary: probability and gradient exactly 0) as long as the sampled token's and at least one other entry of every
 *                 unmasked row is finite; +inf and NaN are not accepted (results unspecified).
 *   targets       [T] int32, the sampled token y_r
 *   mask          [T] uint8, non-zero = the token counts; NULL = all ones.  Masked rows of
 *                 logits are never read.
 *   behav_logp    [T] float, log mu(y_t|.) stored by the behaviour policy at sampling time
 *   rewards       [N] float
 *   group_offsets [K+1] int32 (see rapid_group_advantage)
 *   dlogits       [T, ld] out, same dtype and pitch as logits; may be the SAME buffer as logits
 *                 (in place).  Partial overlap is not allowed.  Rows that are masked, or whose
 *                 coefficient g_n is zero, are written as zeros.  Columns >= vocab are untouched.
 *   loss          [1] float out
 *   token_logp    [T] float out (0 on masked rows); may be NULL.  token_logp[r] - behav_logp[r] is
 *                 the token-level importance weight in log scale that Sec. 4.3 plots for a single
 *                 generation; stats->n_clipped / N is the clipped share it reports per inner step
 *   adv           [N] float out; may be NULL
 *   stats         out; may be NULL
 *   workspace     rapid_workspace_bytes(desc) bytes, 256-byte aligned
 */
rapid_status_t rapid_pg_loss_fwd_bwd(const rapid_desc_t* desc, const void* logits,
                                     const int32_t* targets, const uint8_t* mask,
                                     const float* behav_logp, const float* rewards,
                                     const int32_t* group_offsets, void* dlogits, float* loss,
                                     float* token_logp, float* adv, rapid_stats_t* stats,
                                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * rapid_pg_loss_fwd_bwd without a caller-provided workspace.  (The paper has no counterpart to
 * this call; it exists for deployment reasons only.)
 *
 * Some users of this library are not in a position to allocate device memory for the workspace:
 * a plug-in inside a host application whose memory pool already owns the whole device and
 * forbids allocations behind its back; a serving or training loop that has handed out its entire
 * memory budget up front and treats any later allocation as a bug; a latency-critical loop that
 * cannot afford the device-wide stall an allocation may cause.  For them the scratch memory is a
 * fixed array of RAPID_NOALLOC_SCRATCH_BYTES inside the library's device image.  Every GPU on
 * which the library is loaded holds that array until the process exits.
 *
 * Arguments and results are exactly those of rapid_pg_loss_fwd_bwd, minus the workspace; the
 * caller still owns and passes every input and output array.
 *
 *   - Limit: the problem must satisfy rapid_workspace_bytes(desc) <= RAPID_NOALLOC_SCRATCH_BYTES
 *     (about 21 bytes per row of the token grid, i.e. up to roughly 199 000 rows).  Anything
 *     larger returns RAPID_ERR_UNSUPPORTED and enqueues nothing; use the workspace form instead.
 *   - The call allocates and frees nothing, on the device or through any library.
 *   - Every call looks up the device address of the array for the caller's current device (a
 *     cudaGetSymbolAddress call) and remembers nothing, so the call stays valid after a
 *     cudaDeviceReset and under whichever context is current.  The FIRST call on a device is the
 *     one that makes the runtime set the array up there: make it, on every device you will use,
 *     before beginning any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left in
 *     it.  Nothing in it needs clearing between calls (each call rewrites what it reads), but two
 *     calls whose GPU work can overlap -- different streams, or different host threads without
 *     ordering between their streams -- race on it and give undefined results.  Serialise them.
 */
#define RAPID_NOALLOC_SCRATCH_BYTES (4u << 20)
rapid_status_t rapid_pg_loss_fwd_bwd_noalloc(const rapid_desc_t* desc, const void* logits,
                                             const int32_t* targets, const uint8_t* mask,
                                             const float* behav_logp, const float* rewards,
                                             const int32_t* group_offsets, void* dlogits,
                                             float* loss, float* token_logp, float* adv,
                                             rapid_stats_t* stats, void* stream);

/*
 * The same path in three steps, for logits that are produced (or fit in memory) only a block of
 * rows at a time.  The order is forced by the data: every generation of a group must have gone
 * through the statistics pass before any of the group's dlogits can be written.
 *
 *   1. rapid_pg_stats_chunk   for every block of rows [row0, row0 + n_rows) of the [T, V] grid,
 *                             in any order, each row exactly once
 *   2. rapid_pg_finalize      once
 *   3. rapid_pg_dlogits_chunk for every block again (the caller re-materialises the same logits)
 *
 * logits_chunk / dlogits_chunk point at row `row0` (so chunk row i is global row row0 + i) and
 * use pitch desc->ld; targets, mask and behav_logp are the FULL [T] arrays.  The workspace is the
 * one from rapid_workspace_bytes(desc), shared by all three steps.  dlogits_chunk may alias
 * logits_chunk.
 *
 * The statistics pass uses ordinary vector loads and has no device-side wait.  The dlogits pass
 * moves data with asynchronous bulk copies and waits for them on barriers; every such wait is
 * bounded (a few seconds).  A wait that gives up never traps: the status word of `stats`
 * (optional; pass the struct that finalize wrote) is raised to RAPID_ERR_TIMEOUT and the affected
 * rows of dlogits are unspecified.
 */
rapid_status_t rapid_pg_stats_chunk(const rapid_desc_t* desc, const void* logits_chunk,
                                    int64_t row0, int64_t n_rows, const int32_t* targets,
                                    const uint8_t* mask, void* workspace, size_t workspace_bytes,
                                    void* stream);

rapid_status_t rapid_pg_finalize(const rapid_desc_t* desc, const float* behav_logp,
                                 const float* rewards, const int32_t* group_offsets, float* loss,
                                 float* token_logp, float* adv, rapid_stats_t* stats,
                                 void* workspace, size_t workspace_bytes, void* stream);

rapid_status_t rapid_pg_dlogits_chunk(const rapid_desc_t* desc, const void* logits_chunk,
                                      void* dlogits_chunk, int64_t row0, int64_t n_rows,
                                      const int32_t* targets, rapid_stats_t* stats,
                                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * rapid_pg_loss_fwd_bwd for logits that lie in page-locked HOST memory (cudaHostAlloc /
 * cudaHostRegister, addressable by the device).  The statistics pass reads the rows straight from
 * host memory over the bus -- masked rows are never transferred -- and leaves a copy of every row it
 * read in `logits_staging`, which the dlogits pass then uses.  This is the one call whose `logits`
 * argument is a host pointer; every other array is device memory as usual.
 *   logits_host     [T, ld] host, page-locked; anything else (pageable host memory, a device
 *                   pointer) returns RAPID_ERR_INVALID_ARG and enqueues nothing
 *   logits_staging  [T, ld] device, same dtype and pitch; rows that are masked are left untouched
 *   dlogits         [T, ld] device; may be logits_staging itself (in place)
 * The other arguments, the results and the workspace are those of rapid_pg_loss_fwd_bwd.
 * (Sec. 3.2 of the paper alternates inference and training on the same devices, so logits normally
 * never leave the GPU; this form exists for pipelines that stage them through the host.)
 */
rapid_status_t rapid_pg_loss_fwd_bwd_hostlogits(const rapid_desc_t* desc, const void* logits_host,
                                                void* logits_staging, const int32_t* targets,
                                                const uint8_t* mask, const float* behav_logp,
                                                const float* rewards, const int32_t* group_offsets,
                                                void* dlogits, float* loss, float* token_logp,
                                                float* adv, rapid_stats_t* stats, void* workspace,
                                                size_t workspace_bytes, void* stream);

/*
 * The on-policy special case in a single pass over the logits.  When the behaviour policy IS the
 * current policy (mu = pi_theta: the first inner step after Algorithm 1 refreshes mu, and every
 * step of the plain policy-gradient baseline) every importance weight is 1, Eq. 3 reduces to
 * Eq. 1 and Eq. 5 to the group advantage of Eq. 2, which needs rewards only.  The coefficient
 * g_n = A_n / Z is then known before any logit is read, so each row is read once from memory
 * (its second sweep is served from L2) and written once:
 *
 *   A_n = R_n - (1/N_k) sum_{n' in group k} R_n'          Eq. 2 (leave-one-out by flag)
 *   loss = - sum_n g_n sum_t m_r log pi_theta(y_t),       Eq. 1
 *   dlogits[r, v] = g_n m_r (softmax(z[r, .])_v - 1[v == y_r])
 *
 * Arguments as for rapid_pg_loss_fwd_bwd, without behav_logp; desc->eta and
 * RAPID_FLAG_OUTER_UNCLIPPED have no effect.  dlogits may be the logits buffer itself.  Rows that
 * are masked are never read; rows of a generation with g_n = 0 (for instance a prompt whose
 * generations all earned the same reward) are read only if token_logp is requested.
 * stats: n_clipped = 0 and both staleness means are 0 by definition.  A bounded wait that gives
 * up raises stats->status to RAPID_ERR_TIMEOUT.
 */
rapid_status_t rapid_pg_loss_onpolicy_fwd_bwd(const rapid_desc_t* desc, const void* logits,
                                              const int32_t* targets, const uint8_t* mask,
                                              const float* rewards, const int32_t* group_offsets,
                                              void* dlogits, float* loss, float* token_logp,
                                              float* adv, rapid_stats_t* stats, void* workspace,
                                              size_t workspace_bytes, void* stream);

/*
 * The fused LM-head form: the logits z = hidden * w_vocab are formed tile by tile on the tensor
 * cores and never written to memory (this form comes from the benchmark definition; in the paper
 * the logits are simply the policy network's output, Sec. 3.1).  Computes the same loss as
 * rapid_pg_loss_fwd_bwd on z, and the gradients with respect to both factors:
 *     dhidden = dlogits * w_vocab^T,      dW = hidden^T * dlogits,
 * where dlogits (as defined at the top of this file) is rounded to bf16 before these two products.
 *
 *   desc        dtype must be RAPID_BF16; desc->ld is the row pitch, in elements, of BOTH w_vocab
 *               and dW (>= vocab, a multiple of 8)
 *   hidden_dim  D, a multiple of 8
 *   hidden      [T, D] bf16, contiguous rows (pitch D), 16-byte aligned.  Every row must be finite,
 *               masked ones too: they enter the products with a zero coefficient (unlike the
 *               logits-in calls, which never read a masked row)
 *   w_vocab     [D, ld] bf16, 16-byte aligned
 *   targets, mask, behav_logp, rewards, group_offsets: as for rapid_pg_loss_fwd_bwd
 *   loss        [1] float out
 *   dhidden     [T, D] bf16 out (pitch D); rows that are masked or have g_n = 0 come out as zeros
 *   dW          [D, ld] float out ([D, ld] bf16 with RAPID_FLAG_HEAD_DW_BF16).  Stores go out in
 *               16-byte units: when vocab is not a multiple of 4 (of 8 for bf16), the columns from
 *               vocab up to the next such multiple are written as zeros; columns beyond that are
 *               untouched
 *   token_logp, adv, stats: optional outputs as for rapid_pg_loss_fwd_bwd
 *   workspace   rapid_fused_head_workspace_bytes(desc, hidden_dim) bytes, 1024-byte aligned.  It
 *               holds, besides the per-row state, two floats per row per 256 vocabulary columns
 *               and a bf16 copy of dlogits for at most 16384 rows at a time ([rows, vocab rounded
 *               up to 64 columns]): the backward part runs over the mini-batch in chunks of that
 *               many rows, dW accumulating from chunk to chunk.  With RAPID_FLAG_HEAD_STORE_LOGITS
 *               the bf16 matrix covers all T rows (it holds the logits first, dlogits afterwards).
 *
 * Tensor-core kernels run for the forward statistics and, per chunk of rows, for dlogits, dhidden
 * and dW (four GEMM-sized contractions over the mini-batch in all; three with
 * RAPID_FLAG_HEAD_STORE_LOGITS, where dlogits come from the stored logits), each a persistent grid
 * with bounded waits: a wait that gives up raises stats->status to RAPID_ERR_TIMEOUT and leaves the
 * outputs unspecified.  Returns RAPID_ERR_CUDA if the driver cannot encode the tensor maps.
 */
rapid_status_t rapid_fused_head_workspace_bytes(const rapid_desc_t* desc, int32_t hidden_dim,
                                                size_t* bytes);

rapid_status_t rapid_pg_loss_fused_head(const rapid_desc_t* desc, int32_t hidden_dim,
                                        const void* hidden, const void* w_vocab,
                                        const int32_t* targets, const uint8_t* mask,
                                        const float* behav_logp, const float* rewards,
                                        const int32_t* group_offsets, float* loss, void* dhidden,
                                        void* dW, float* token_logp, float* adv,
                                        rapid_stats_t* stats, void* workspace,
                                        size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RAPID_PG_H */
