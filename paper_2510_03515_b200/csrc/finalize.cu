// Between the two passes over the logits: per-generation sums of token log-probabilities
// (the generation-level importance weight of Sec. 4.3), the clipped weights and the group
// advantage (Eq. 5; Eq. 2 / Eq. 4 as special cases; leave-one-out by flag), the per-generation
// coefficient of Eq. 3, the scalar loss and the side statistics.  Everything here is double and
// touches O(T) scalars, so it is launch-latency only.
//
// The group sums run in index order with explicit round-to-nearest multiplies and adds (no
// fused multiply-add), so rapid_group_advantage is bit-identical to the plain definition.
#include "rapid_common.cuh"

namespace rapid {

namespace {

constexpr int kSeqThreads = 256;
constexpr int kFinThreads = 256;

// ---- step 2: one CTA per generation --------------------------------------------------------------

__global__ void __launch_bounds__(kSeqThreads)
seq_reduce_kernel(int seq_len, const float* __restrict__ behav_logp,
                  float* __restrict__ token_logp_out, Workspace ws) {
    __shared__ double sh_a[kSeqThreads / 32], sh_b[kSeqThreads / 32];
    __shared__ int sh_c[kSeqThreads / 32], sh_d[kSeqThreads / 32];
    const int n = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t base = (int64_t)n * seq_len;
    double s = 0.0, S = 0.0;
    int cnt = 0, bad = 0;
    for (int t = tid; t < seq_len; t += kSeqThreads) {
        const int64_t r = base + t;
        const uint8_t st = ws.row_state[r];
        double lp = 0.0;
        if (st == ROW_OK) {
            lp = ws.token_logp[r];
            if (behav_logp) s += lp - (double)behav_logp[r];  // no behaviour policy: on-policy, s_n = 0
            S += lp;
            cnt += 1;
        } else if (st == ROW_BAD_TOKEN) {
            bad += 1;
        }
        if (token_logp_out) token_logp_out[r] = (float)lp;
    }
    s = warp_sum(s);
    S = warp_sum(S);
    cnt = warp_sum(cnt);
    bad = warp_sum(bad);
    if (lane == 0) {
        sh_a[warp] = s;
        sh_b[warp] = S;
        sh_c[warp] = cnt;
        sh_d[warp] = bad;
    }
    __syncthreads();
    if (tid == 0) {
        double a = 0.0, b = 0.0;
        int c = 0, d = 0;
        for (int w = 0; w < kSeqThreads / 32; ++w) {
            a += sh_a[w];
            b += sh_b[w];
            c += sh_c[w];
            d += sh_d[w];
        }
        ws.seq_log_ratio[n] = a;
        ws.seq_logp[n] = b;
        ws.seq_tokens[n] = c;
        ws.seq_bad[n] = d;
    }
}

// ---- steps 3-5: one CTA ------------------------------------------------------------------------

__device__ __forceinline__ double weight_of(const double* slr, int n, uint32_t flags) {
    if (!slr) return 1.0;
    return (flags & RAPID_FLAG_ADV_INPUT_IS_WEIGHT) ? slr[n] : exp(slr[n]);
}
__device__ __forceinline__ double clip_w(double w, double eta) { return (w < eta) ? w : eta; }

template <typename T>
__device__ __forceinline__ T block_sum(T v, T* sh) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) sh[warp] = v;
    __syncthreads();
    T tot = 0;
    for (int w = 0; w < kFinThreads / 32; ++w) tot += sh[w];
    return tot;
}

// full == true : the loss path (uses the workspace's per-generation sums, writes coefficients).
// full == false: rapid_group_advantage on caller-provided log-ratios / weights.
template <bool full>
__global__ void __launch_bounds__(kFinThreads)
finalize_kernel(int n_seq, int n_groups, double eta, double norm_z, uint32_t flags,
                const float* __restrict__ rewards, const double* __restrict__ slr_in,
                const int32_t* __restrict__ group_offsets, float* __restrict__ loss_out,
                float* __restrict__ adv_out, double* __restrict__ clipped_out,
                rapid_stats_t* __restrict__ stats_out, Workspace ws) {
    __shared__ int sh_bad_groups;
    __shared__ int sh_empty;
    __shared__ double sh_d[kFinThreads / 32];
    __shared__ long long sh_l[kFinThreads / 32];
    __shared__ int sh_i[kFinThreads / 32];
    const int tid = threadIdx.x;
    const double* slr = full ? ws.seq_log_ratio : slr_in;

    if (tid == 0) {
        sh_bad_groups = 0;
        sh_empty = 0;
    }
    __syncthreads();
    // group_offsets must be a monotone cover of [0, N)
    for (int k = tid; k <= n_groups; k += kFinThreads) {
        const int o = group_offsets[k];
        bool bad = (k == 0 && o != 0) || (k == n_groups && o != n_seq) || o < 0 || o > n_seq;
        if (k < n_groups) {
            const int o1 = group_offsets[k + 1];
            if (o1 < o) bad = true;
            if (o1 == o) atomicAdd(&sh_empty, 1);
        }
        if (bad) atomicAdd(&sh_bad_groups, 1);
    }
    __syncthreads();
    const bool groups_ok = (sh_bad_groups == 0);

    if (!groups_ok) {
        const float nanf_ = __int_as_float(0x7fc00000);
        for (int n = tid; n < n_seq; n += kFinThreads) {
            if (adv_out) adv_out[n] = nanf_;
            if (clipped_out) clipped_out[n] = (double)nanf_;
            if (full) {
                ws.coef[n] = 0.0;
                ws.coef_log2[n] = -INFINITY;
                ws.adv[n] = (double)nanf_;
            }
        }
        if (tid == 0) {
            if (loss_out) *loss_out = nanf_;
            rapid_stats_t st;
            st.n_tokens = 0;
            st.n_clipped = 0;
            st.n_bad_token = 0;
            st.n_empty_group = 0;
            st.status = RAPID_ERR_INVALID_ARG;
            st.mean_log_cw = (double)nanf_;
            st.mean_abs_log_cw = (double)nanf_;
            st.loss = (double)nanf_;
            if (stats_out) *stats_out = st;
            if (full) *ws.stats = st;
        }
        return;
    }

    // step 3, one thread per generation: the weight and its clipped value
    for (int n = tid; n < n_seq; n += kFinThreads) {
        const double w = weight_of(slr, n, flags);
        const double c = clip_w(w, eta);
        if (full) {
            ws.weight[n] = w;
            ws.clipped_w[n] = c;
        }
        if (clipped_out) clipped_out[n] = c;
    }
    __syncthreads();
    auto clipped = [&](int q) -> double {
        if (full) return ws.clipped_w[q];
        return clipped_out ? clipped_out[q] : clip_w(weight_of(slr, q, flags), eta);
    };
    // step 4: every sum runs over the group's members in index order, exactly as the definition reads
    if (!(flags & RAPID_FLAG_LEAVE_ONE_OUT)) {
        // one thread per group: the baseline is shared by its members
        for (int k = tid; k < n_groups; k += kFinThreads) {
            const int lo = group_offsets[k], hi = group_offsets[k + 1];
            const int Nk = hi - lo;
            if (Nk == 0) continue;
            double csum = 0.0;
            for (int n = lo; n < hi; ++n) csum = __dadd_rn(csum, __dmul_rn(clipped(n), (double)rewards[n]));
            const double base = __ddiv_rn(csum, (double)Nk);
            for (int n = lo; n < hi; ++n) {
                const double a = __dsub_rn((double)rewards[n], base);
                if (full) ws.adv[n] = a;
                if (adv_out) adv_out[n] = (float)a;
            }
        }
    } else {
        // leave-one-out: every member has its own sum over the others, so one thread per MEMBER (a
        // single group of thousands of generations -- the single-path baseline -- would otherwise
        // leave N_k^2 additions to one thread).  The member's group is found by bisection.
        for (int n = tid; n < n_seq; n += kFinThreads) {
            int a0 = 0, a1 = n_groups;  // the last k with group_offsets[k] <= n; empty groups before it are skipped
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
                if (q != n) others = __dadd_rn(others, __dmul_rn(clipped(q), (double)rewards[q]));
            double a;
            if (flags & RAPID_FLAG_LOO_LITERAL_DIVISOR) a = __dsub_rn(R, __ddiv_rn(others, (double)Nk));
            else if (Nk > 1) a = __dsub_rn(R, __ddiv_rn(others, (double)(Nk - 1)));
            else a = R;
            if (full) ws.adv[n] = a;
            if (adv_out) adv_out[n] = (float)a;
        }
    }
    __syncthreads();

    // step 5 and the statistics
    long long tokens = 0;
    int bad_tok = 0;
    if (full) {
        for (int n = tid; n < n_seq; n += kFinThreads) {
            tokens += ws.seq_tokens[n];
            bad_tok += ws.seq_bad[n];
        }
    }
    tokens = block_sum<long long>(tokens, sh_l);
    bad_tok = block_sum<int>(bad_tok, sh_i);
    const double Z = (flags & RAPID_FLAG_NORM_GIVEN)    ? norm_z
                     : (flags & RAPID_FLAG_NORM_TOKENS) ? (double)tokens
                                                        : (double)n_seq;
    const double log_eta = log(eta);

    double loss = 0.0, sum_log = 0.0, sum_abs = 0.0;
    int n_clip = 0;
    for (int n = tid; n < n_seq; n += kFinThreads) {
        const double w = full ? ws.weight[n] : weight_of(slr, n, flags);
        if (w > eta) n_clip += 1;
        double lc;
        if (!slr)
            lc = 0.0;
        else if (!full && (flags & RAPID_FLAG_ADV_INPUT_IS_WEIGHT))
            lc = log(clip_w(w, eta));
        else
            lc = (slr[n] < log_eta) ? slr[n] : log_eta;
        sum_log += lc;
        sum_abs += fabs(lc);
        if (full) {
            const double chat = (flags & RAPID_FLAG_OUTER_UNCLIPPED) ? w : ws.clipped_w[n];
            const double g = (Z > 0.0) ? chat * ws.adv[n] / Z : 0.0;
            ws.coef[n] = g;
            ws.coef_log2[n] = (g != 0.0) ? log2(fabs(g)) : -INFINITY;
            loss -= g * ws.seq_logp[n];
        }
    }
    loss = block_sum<double>(loss, sh_d);
    sum_log = block_sum<double>(sum_log, sh_d);
    sum_abs = block_sum<double>(sum_abs, sh_d);
    n_clip = block_sum<int>(n_clip, sh_i);
    if (tid == 0) {
        rapid_stats_t st;
        st.n_tokens = tokens;
        st.n_clipped = n_clip;
        st.n_bad_token = bad_tok;
        st.n_empty_group = sh_empty;
        st.status = RAPID_OK;
        st.mean_log_cw = sum_log / (double)n_seq;
        st.mean_abs_log_cw = sum_abs / (double)n_seq;
        st.loss = full ? loss : 0.0;
        if (stats_out) *stats_out = st;
        if (full) {
            *ws.stats = st;
            if (loss_out) *loss_out = (float)loss;
        }
    }
}

}  // namespace

cudaError_t launch_seq_reduce(const rapid_desc_t& d, const float* behav_logp, float* token_logp_out,
                              const Workspace& ws, cudaStream_t stream) {
    seq_reduce_kernel<<<d.n_seq, kSeqThreads, 0, stream>>>(d.seq_len, behav_logp, token_logp_out, ws);
    return cudaGetLastError();
}

cudaError_t launch_finalize(const rapid_desc_t& d, const float* rewards,
                            const int32_t* group_offsets, float* loss, float* adv,
                            rapid_stats_t* stats_out, const Workspace& ws, cudaStream_t stream) {
    finalize_kernel<true><<<1, kFinThreads, 0, stream>>>(d.n_seq, d.n_groups, d.eta, d.norm_z, d.flags, rewards,
                                                        nullptr, group_offsets, loss, adv, nullptr,
                                                        stats_out, ws);
    return cudaGetLastError();
}

cudaError_t launch_group_advantage(const rapid_desc_t& d, const float* rewards,
                                   const double* seq_log_ratio, const int32_t* group_offsets,
                                   float* adv, double* clipped_w, rapid_stats_t* stats_out,
                                   cudaStream_t stream) {
    Workspace none = {};
    finalize_kernel<false><<<1, kFinThreads, 0, stream>>>(d.n_seq, d.n_groups, d.eta, d.norm_z, d.flags,
                                                         rewards, seq_log_ratio, group_offsets,
                                                         nullptr, adv, clipped_w, stats_out, none);
    return cudaGetLastError();
}

}  // namespace rapid
