// Device-side control of the loop: LM-head finish (bias, argmax), end of a draft
// step, block test of the pre-verification (Algorithm 1), acceptance and cache
// rollback (Eq. 5).  All decisions are taken on the device from SeqState.
#pragma once
#include "common.cuh"

constexpr int HEAD_THREADS = 1024;

struct Top2 {
    float v1; int i1; float v2;
};

__device__ __forceinline__ Top2 top2_merge(Top2 a, Top2 b) {
    // larger value wins; equal values keep the lower index
    Top2 r;
    const bool a_first = (a.v1 > b.v1) || (a.v1 == b.v1 && a.i1 <= b.i1);
    if (a_first) { r.v1 = a.v1; r.i1 = a.i1; r.v2 = fmaxf(a.v2, b.v1); }
    else { r.v1 = b.v1; r.i1 = b.i1; r.v2 = fmaxf(b.v2, a.v1); }
    return r;
}

__device__ __forceinline__ Top2 block_top2(Top2 t, Top2 *sm) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Top2 u;
        u.v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
        u.i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
        u.v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
        t = top2_merge(t, u);
    }
    if (lane == 0) sm[w] = t;
    __syncthreads();
    if (w == 0) {
        Top2 u = lane < nw ? sm[lane] : Top2{-INFINITY, 0x7fffffff, -INFINITY};
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            Top2 x;
            x.v1 = __shfl_xor_sync(0xffffffffu, u.v1, o);
            x.i1 = __shfl_xor_sync(0xffffffffu, u.i1, o);
            x.v2 = __shfl_xor_sync(0xffffffffu, u.v2, o);
            u = top2_merge(u, x);
        }
        if (lane == 0) sm[0] = u;
    }
    __syncthreads();
    return sm[0];
}

// Sums the LM-head partials of one row, adds the planted bias on succ[input
// token], stores the logits where the stage wants them, and finds the argmax
// (lowest index on ties) with the gap to the runner-up.
// kind DRAFT: only the last active row of each sequence matters (it emits y_i);
// its logits go to draft_logits[seq][gamma].  kind VERIFY: every active row j
// goes to verify_logits[seq][j].  kind AR: row 0 to verify_logits[seq][0].
__global__ void __launch_bounds__(HEAD_THREADS) k_head_finish(DevPtrs d, ModelDev m, Geom g, int kind, int S) {
    __shared__ Top2 sm[32];
    const int r = blockIdx.x, s = r / g.rps, j = r - s * g.rps;
    if (d.row_pos[r] < 0) return;
    const int V = m.cfg.vocab;
    float *dst;
    if (kind == KIND_DRAFT) {
        if (j != d.n_rows[s] - 1) return;
        dst = d.draft_logits + ((size_t)s * d.gamma_cap + d.st[s].gamma) * V;
    } else {
        dst = d.verify_logits + ((size_t)s * (d.gamma_cap + 1) + j) * V;
    }
    const size_t sstride = (size_t)g.nt * 8 * V;
    const float *p = d.part + (size_t)r * V;
    const int bias_at = m.succ ? m.succ[d.row_tok[r]] : -1;
    Top2 t{-INFINITY, 0x7fffffff, -INFINITY};
    for (int v = threadIdx.x; v < V; v += blockDim.x) {
        float val = 0.f;
        for (int ss = 0; ss < S; ++ss) val += p[ss * sstride + v];
        if (v == bias_at) val += d.succ_bias;
        dst[v] = val;
        if (val > t.v1) { t.v2 = t.v1; t.v1 = val; t.i1 = v; }
        else if (val > t.v2) t.v2 = val;
    }
    t = block_top2(t, sm);
    if (threadIdx.x == 0) { d.row_arg[r] = t.i1; d.row_margin[r] = t.v1 - t.v2; }
}

// End of one draft forward (Eq. 6): y_i, h_i queued for M_B, cache length.
__global__ void __launch_bounds__(256) k_draft_end(DevPtrs d, Geom g, int dm) {
    const int s = blockIdx.x;
    SeqState &st = d.st[s];
    const int n_in = d.n_rows[s];
    if (n_in == 0) return;
    const int r_last = s * g.rps + n_in - 1;
    const int gamma = st.gamma, n_pend = st.n_pend;
    for (int jj = 0; jj < n_in; ++jj) {
        const float *h = d.hidden + (size_t)(s * g.rps + jj) * dm;
        float *dst = d.hpend + ((size_t)s * (d.block_b + 1) + n_pend + jj) * dm;
        for (int i = threadIdx.x; i < dm; i += blockDim.x) dst[i] = h[i];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int jj = 0; jj < n_in; ++jj)
            d.hpend_e[s * (d.block_b + 1) + n_pend + jj] = (jj == n_in - 1) ? gamma + 1 : 0;
        d.y[(size_t)s * d.gamma_cap + gamma] = d.row_arg[r_last];
        st.n_pend = n_pend + n_in;
        st.gamma = gamma + 1;
        st.len_D += n_in;
        st.n_draft_fwd += 1;
    }
}

// End of a pre-verification call (Eq. 7 + block test): alpha_hat of the new
// drafts from the 2-way head, block statistic, stop decision, threshold growth.
__global__ void __launch_bounds__(256) k_mb_end(DevPtrs d, ModelDev m, Geom g) {
    __shared__ float red[33];
    const int s = blockIdx.x;
    SeqState &st = d.st[s];
    const int n = d.n_rows[s];
    if (n == 0) return;
    const int dm = m.cfg.d_model;
    for (int j = 0; j < n; ++j) {
        const int e = d.row_tok[s * g.rps + j];
        if (e == 0) continue;
        const float *h = d.hidden + (size_t)(s * g.rps + j) * dm;
        float z0 = 0.f, z1 = 0.f;
        for (int i = threadIdx.x; i < dm; i += blockDim.x) {
            const float hv = h[i];
            z0 += hv * __bfloat162float(m.head_b[i]);
            z1 += hv * __bfloat162float(m.head_b[dm + i]);
        }
        z0 = block_sum(z0, red);
        z1 = block_sum(z1, red);
        if (threadIdx.x == 0) d.alpha[(size_t)s * d.gamma_cap + e - 1] = 1.f / (1.f + expf(z0 - z1));
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int b = d.block_b, gamma = st.gamma;
        const float *ab = d.alpha + (size_t)s * d.gamma_cap + (gamma - b);
        float stat;
        if (d.criterion == 1) { stat = ab[0]; for (int i = 1; i < b; ++i) stat = fminf(stat, ab[i]); }
        else if (d.criterion == 2) stat = ab[b - 1];
        else { stat = 0.f; for (int i = 0; i < b; ++i) stat += ab[i]; stat /= (float)b; }
        int stop = 0;
        if (st.t0 >= 0.f && stat <= st.t_k) stop = 1;
        if (gamma + b > st.gamma_max) stop = 1;
        if (stop) st.drafting = 0;
        else { st.t_k = st.t_k * d.rho; st.k_round += 1; }
        st.len_B += n;
        st.n_pend = 0;
        st.n_mb_calls += 1;
    }
}

// Greedy acceptance (Eq. 5 with one-hot distributions), commit, rollback, logs.
__global__ void k_accept_greedy(DevPtrs d, Geom g) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= g.batch) return;
    SeqState &st = d.st[s];
    if (!st.active || st.finished || d.n_rows[s] == 0) return;
    const int gamma = st.gamma, P = st.P;
    const int32_t *y = d.y + (size_t)s * d.gamma_cap;
    const int32_t *arg = d.row_arg + s * g.rps;
    int n = 0;
    while (n < gamma && y[n] == arg[n]) ++n;
    const int next = arg[n];
    int32_t *x = d.x + (size_t)s * d.max_ctx;
    for (int i = 0; i < n; ++i) x[P + i] = y[i];
    x[P + n] = next;
    st.P = P + n + 1;
    st.len_T = P + n;                                     // verify wrote rows P-1 .. P-1+gamma
    const int keep = P - 1 + (n + 1 < gamma ? n + 1 : gamma);   // the draft never processed y_gamma
    st.len_D = keep;
    st.len_B = keep;
    st.last_n = n; st.last_next = next;
    if (st.n_steps < d.max_steps) {
        d.draft_len[(size_t)s * d.max_steps + st.n_steps] = gamma;
        d.accept_len[(size_t)s * d.max_steps + st.n_steps] = n;
    }
    st.n_steps += 1;
    st.n_target_fwd += 1;
    st.gamma = 0; st.k_round = 0; st.t_k = st.t0; st.drafting = 1; st.n_pend = 0;
    if (st.P - st.n_prompt >= st.max_new) { st.finished = 1; st.drafting = 0; }
}

// End of one autoregressive target step (Eq. 1).
__global__ void k_ar_end(DevPtrs d, Geom g) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= g.batch) return;
    SeqState &st = d.st[s];
    if (!st.active || st.finished || d.n_rows[s] == 0) return;
    d.x[(size_t)s * d.max_ctx + st.P] = d.row_arg[s * g.rps];
    st.P += 1;
    st.len_T += 1;
    st.n_target_fwd += 1;
    st.n_steps += 1;
    if (st.P - st.n_prompt >= st.max_new) st.finished = 1;
}

// After a prefill chunk: nothing to decide, the caches grow by the rows written.
__global__ void k_prefill_end(DevPtrs d, Geom g, int which) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= g.batch) return;
    SeqState &st = d.st[s];
    if (!st.active) return;
    const int n = d.n_rows[s];
    if (which == PACER_TARGET) st.len_T += n;
    else if (which == PACER_DRAFT) st.len_D += n;
    else st.len_B += n;
}
