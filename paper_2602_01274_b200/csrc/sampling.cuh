// Seeded sampling at temperature 1: counter-based uniforms (Philox4x32-10, Salmon
// et al., "Parallel random numbers: as easy as 1, 2, 3"), Gumbel-max draws from
// logits, and the acceptance rule of speculative sampling (Eq. 5; Algorithm 1's
// accept / resample part) with commit and cache rollback.
//
// One uniform belongs to (vocabulary index v, absolute position, sequence, tag):
// counter = (v / 4, position, sequence, tag), key = the seed's two halves, word
// v % 4 of the output block, u = ((word >> 8) + 0.5) * 2^-24 in (0, 1).
// Gumbel noise -log(-log u) is evaluated in fp64 (u can be within 2^-25 of 1).
#pragma once
#include "common.cuh"
#include "control.cuh"

enum { TAG_DRAFT = 1, TAG_ACCEPT = 2, TAG_NEXT = 3 };

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                              uint32_t (&out)[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
        const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = h1 ^ c1 ^ k0, n2 = h0 ^ c3 ^ k1;
        c0 = n0; c1 = l1; c2 = n2; c3 = l0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

__device__ __forceinline__ double uniform01(uint64_t seed, uint32_t v, uint32_t pos, uint32_t seq, uint32_t tag) {
    uint32_t o[4];
    philox4x32_10(v >> 2, pos, seq, tag, (uint32_t)seed, (uint32_t)(seed >> 32), o);
    const uint32_t w = (v & 3) == 0 ? o[0] : (v & 3) == 1 ? o[1] : (v & 3) == 2 ? o[2] : o[3];
    return ((double)(w >> 8) + 0.5) * (1.0 / 16777216.0);
}

__device__ __forceinline__ double gumbel_noise(uint64_t seed, uint32_t v, uint32_t pos, uint32_t seq, uint32_t tag) {
    return -log(-log(uniform01(seed, v, pos, seq, tag)));
}

struct BestD {
    double v; int i;
};
__device__ __forceinline__ BestD best_merge(BestD a, BestD b) {       // larger value; equal values keep the lower index
    return (a.v > b.v || (a.v == b.v && a.i <= b.i)) ? a : b;
}

// Block-wide arg-max of a per-thread candidate; every thread gets the result.
// sm: at least blockDim.x / 32 entries.  All threads of the block must call it.
__device__ __forceinline__ BestD block_best(BestD t, BestD *sm, bool named_barrier) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        BestD u;
        u.v = __shfl_xor_sync(0xffffffffu, t.v, o);
        u.i = __shfl_xor_sync(0xffffffffu, t.i, o);
        t = best_merge(t, u);
    }
    const int nw = named_barrier ? 8 : (blockDim.x >> 5);
    if (named_barrier) asm volatile("bar.sync 1, 256;" ::: "memory"); else __syncthreads();
    if (lane == 0) sm[w] = t;
    if (named_barrier) asm volatile("bar.sync 1, 256;" ::: "memory"); else __syncthreads();
    BestD r = sm[0];
    for (int i = 1; i < nw; ++i) r = best_merge(r, sm[i]);
    if (named_barrier) asm volatile("bar.sync 1, 256;" ::: "memory"); else __syncthreads();
    return r;
}

// A draw from softmax(logits) by the Gumbel-max rule: argmax_v(logit_v + G_v).
// nthreads threads (threadIdx.x < nthreads) walk the row; result in every thread.
__device__ __forceinline__ int gumbel_argmax(const float *logits, int V, uint64_t seed, int pos, int seq, int tag, int nthreads,
                                             BestD *sm, bool named_barrier) {
    BestD t{-INFINITY, 0x7fffffff};
    for (int v = threadIdx.x; v < V; v += nthreads) {
        const double s = (double)__ldcg(logits + v) + gumbel_noise(seed, (uint32_t)v, (uint32_t)pos, (uint32_t)seq, (uint32_t)tag);
        if (s > t.v) { t.v = s; t.i = v; }
    }
    return block_best(t, sm, named_barrier).i;
}

// Block-wide sum of doubles (plain __syncthreads version, for the acceptance kernel).
__device__ __forceinline__ double block_sum_d(double v, double *sm) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = v;
    __syncthreads();
    double s = 0.0;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) s += sm[i];
    __syncthreads();
    return s;
}
__device__ __forceinline__ double block_max_d(double v, double *sm) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = v;
    __syncthreads();
    double s = -INFINITY;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) s = fmax(s, sm[i]);
    __syncthreads();
    return s;
}

// log-sum-exp of one logits row (fp64 accumulation), result in every thread.
__device__ __forceinline__ double block_lse(const float *row, int V, double *sm) {
    double mx = -INFINITY;
    for (int v = threadIdx.x; v < V; v += blockDim.x) mx = fmax(mx, (double)__ldcg(row + v));
    mx = block_max_d(mx, sm);
    double s = 0.0;
    for (int v = threadIdx.x; v < V; v += blockDim.x) s += exp((double)__ldcg(row + v) - mx);
    s = block_sum_d(s, sm);
    return mx + log(s);
}

constexpr int ACCEPT_THREADS = 1024;

// Acceptance by rejection sampling (Eq. 5), one block per sequence: draft y_i is
// kept while r_i <= p_i(y_i) / q_i(y_i) (tested as log r <= log p - log q); on the
// first rejection the next token is drawn from norm(max(0, p - q)) of that
// position, when all are kept from p_{gamma+1}; then commit, cache rollback, logs.
__global__ void __launch_bounds__(ACCEPT_THREADS) k_accept_sample(DevPtrs d, Geom g, int V) {
    __shared__ double smd[32];
    __shared__ BestD smb[32];
    const int s = blockIdx.x;
    SeqState &st = d.st[s];
    if (!st.active || st.finished || d.n_rows[s] == 0) return;
    const int gamma = st.gamma, P = st.P;
    const uint64_t seed = st.seed;
    const int32_t *y = d.y + (size_t)s * d.gamma_cap;
    const float *plog = d.verify_logits + (size_t)s * (d.gamma_cap + 1) * V;
    const float *qlog = d.draft_logits + (size_t)s * d.gamma_cap * V;
    int n = 0;
    double lsp = 0.0, lsq = 0.0;
    for (; n < gamma; ++n) {
        const float *p = plog + (size_t)n * V, *q = qlog + (size_t)n * V;
        lsp = block_lse(p, V, smd);
        lsq = block_lse(q, V, smd);
        const double lp = (double)__ldcg(p + y[n]) - lsp, lq = (double)__ldcg(q + y[n]) - lsq;
        const double lr = log(uniform01(seed, 0u, (uint32_t)(P + n), (uint32_t)s, TAG_ACCEPT));
        if (lr > lp - lq) break;                     // r > p / q: reject (the same value in every thread)
    }
    int next;
    if (n == gamma) {
        next = gumbel_argmax(plog + (size_t)gamma * V, V, seed, P + gamma, s, TAG_NEXT, ACCEPT_THREADS, smb, false);
    } else {
        const float *p = plog + (size_t)n * V, *q = qlog + (size_t)n * V;
        BestD t{-INFINITY, 0x7fffffff};
        for (int v = threadIdx.x; v < V; v += ACCEPT_THREADS) {
            const double res = exp((double)__ldcg(p + v) - lsp) - exp((double)__ldcg(q + v) - lsq);
            if (!(res > 0.0)) continue;
            const double sc = log(res) + gumbel_noise(seed, (uint32_t)v, (uint32_t)(P + n), (uint32_t)s, TAG_NEXT);
            if (sc > t.v) { t.v = sc; t.i = v; }
        }
        t = block_best(t, smb, false);
        next = t.i;
        if (t.i == 0x7fffffff) {                     // p == q exactly: cannot be rejected in exact arithmetic
            BestD a{-INFINITY, 0x7fffffff};
            for (int v = threadIdx.x; v < V; v += ACCEPT_THREADS) {
                const double pv = (double)__ldcg(p + v);
                if (pv > a.v) { a.v = pv; a.i = v; }
            }
            next = block_best(a, smb, false).i;
        }
    }
    if (threadIdx.x == 0) commit_step(d, st, s, n, next);
}
