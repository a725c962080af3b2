// Device-side control of the loop: top-2 reductions for the LM head, and the
// acceptance + cache rollback kernel (Eq. 5).  The ends of the draft /
// pre-verification / autoregressive forwards are tails of the forward kernel.
// All decisions are taken on the device from SeqState.
#pragma once
#include "common.cuh"

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

// Commit of one step (Algorithm 1, after Eq. 5): [y_1..y_n, next] joins the accepted tokens, the three caches are
// cut back to the accepted rows, the per-step state restarts, (gamma, n) is logged.  One thread per sequence.
__device__ __forceinline__ void commit_step(const DevPtrs &d, SeqState &st, int s, int n, int next) {
    const int gamma = st.gamma, P = st.P;
    const int32_t *y = d.y + (size_t)s * d.gamma_cap;
    int32_t *x = d.x + (size_t)s * d.max_ctx;
    for (int i = 0; i < n; ++i) x[P + i] = y[i];
    x[P + n] = next;
    st.P = P + n + 1;
    st.len_T = P + n;                                     // verify wrote rows P-1 .. P-1+gamma
    const int keep = P - 1 + (n + 1 < gamma ? n + 1 : gamma);   // the draft never processed y_gamma
    if (keep < st.len_D) st.len_D = keep;                 // (a step without drafts leaves the draft cache as it is)
    st.len_B = st.len_D;
    st.last_n = n; st.last_next = next;
    if (st.n_steps < d.max_steps) {
        d.draft_len[(size_t)s * d.max_steps + st.n_steps] = gamma;
        d.accept_len[(size_t)s * d.max_steps + st.n_steps] = n;
    }
    st.n_steps += 1;
    st.n_target_fwd += 1;
    st.gamma = 0; st.k_round = 0; st.t_k = st.t0; st.drafting = 1; st.n_pend = 0;
    if (st.sched) {                                       // the next step's prescribed window
        int w = d.sched_win[(size_t)s * d.max_steps + (st.n_steps < st.n_sched ? st.n_steps : st.n_sched - 1)];
        if (w > d.gamma_cap) w = d.gamma_cap;
        if (w == 0 && st.P - st.len_D >= d.sched_rows) w = 1;   // the draft's backlog must fit one forward
        st.gamma_max = w;
        st.drafting = w > 0;
    }
    if (st.P - st.n_prompt >= st.max_new) { st.finished = 1; st.drafting = 0; }
}

// Greedy acceptance (Eq. 5 with one-hot distributions) of sequence s: the longest prefix of the drafts that equals
// the target's arg-max tokens, then the commit.  One thread.
__device__ __forceinline__ void accept_greedy_seq(const DevPtrs &d, const Geom &g, int s) {
    SeqState &st = d.st[s];
    if (!st.active || st.finished || d.n_rows[s] == 0) return;
    const int gamma = st.gamma;
    const int32_t *y = d.y + (size_t)s * d.gamma_cap;
    const int32_t *arg = d.row_arg + s * g.rps;
    int n = 0;
    while (n < gamma && y[n] == arg[n]) ++n;
    commit_step(d, st, s, n, arg[n]);
}

// The same as a kernel of its own, for the stage-by-stage interface (the whole-loop entry points take the
// decision in the tail of the verify forward).
__global__ void k_accept_greedy(DevPtrs d, Geom g) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s < g.batch) accept_greedy_seq(d, g, s);
}
