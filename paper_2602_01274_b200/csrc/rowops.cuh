// Row-wise kernels between the GEMMs: row set-up + embedding gather, RMSNorm with
// residual add and split-K reduction, rotary embedding + KV append, SwiGLU.
// One block per row; rows that are inactive in this forward return at once.
#pragma once
#include "common.cuh"

constexpr int ROW_THREADS = 256;

struct RowDesc {
    int active, pos, tok;
};

// Which cache position and input a row of a forward has, derived from the
// sequence state alone (device-side control: no host value is involved).
__device__ __forceinline__ RowDesc row_desc(int kind, const DevPtrs &d, int s, int j, int aux) {
    const SeqState &st = d.st[s];
    RowDesc r;
    r.active = 0; r.pos = -1; r.tok = 0;
    if (!st.active) return r;
    switch (kind) {
        case KIND_DRAFT: {
            if (!st.drafting || st.finished) break;
            if (st.gamma == 0) {
                int n_in = st.P - st.len_D;                  // 1, or 2 after a fully accepted step
                if (j < n_in) { r.active = 1; r.pos = st.len_D + j; r.tok = d.x[(size_t)s * d.max_ctx + r.pos]; }
            } else if (j == 0) {
                r.active = 1; r.pos = st.len_D; r.tok = d.y[(size_t)s * d.gamma_cap + st.gamma - 1];
            }
            break;
        }
        case KIND_VERIFY: {
            if (st.finished) break;
            if (j <= st.gamma) {
                r.active = 1; r.pos = st.P - 1 + j;
                r.tok = j == 0 ? d.x[(size_t)s * d.max_ctx + st.P - 1] : d.y[(size_t)s * d.gamma_cap + j - 1];
            }
            break;
        }
        case KIND_AR: {
            if (st.finished) break;
            if (j == 0) { r.active = 1; r.pos = st.P - 1; r.tok = d.x[(size_t)s * d.max_ctx + st.P - 1]; }
            break;
        }
        case KIND_PREFILL:
        case KIND_PREFILL_B: {
            int p = aux + j;
            if (p < st.n_prompt - 1) { r.active = 1; r.pos = p; r.tok = d.x[(size_t)s * d.max_ctx + p]; }
            break;
        }
        case KIND_MB: {
            if (st.finished) break;
            if (j < st.n_pend) { r.active = 1; r.pos = st.len_B + j; r.tok = d.hpend_e[s * (d.block_b + 1) + j]; }
            break;
        }
    }
    return r;
}

// RMSNorm of one row held in global fp32 memory; writes bf16 in fragment order
// and optionally the fp32 result.
__device__ __forceinline__ void rmsnorm_row(const float *xrow, const bf16 *gain, int dmodel, float eps, int r, int nt,
                                            bf16 *xn, float *hidden_row, float *red) {
    float ss = 0.f;
    for (int i = threadIdx.x; i < dmodel; i += blockDim.x) { float v = xrow[i]; ss += v * v; }
    ss = block_sum(ss, red);
    const float inv = rsqrtf(ss / (float)dmodel + eps);
    for (int i = threadIdx.x; i < dmodel; i += blockDim.x) {
        float v = xrow[i] * inv * __bfloat162float(gain[i]);
        xn[xfrag_index(r, i, nt)] = __float2bfloat16(v);
        if (hidden_row) hidden_row[i] = v;
    }
}

// First kernel of every forward: row descriptors, input rows (embedding gather,
// or h + e for the pre-verification model), first RMSNorm.
__global__ void __launch_bounds__(ROW_THREADS) k_begin(DevPtrs d, ModelDev m, Geom g, int kind, int aux) {
    __shared__ float red[33];
    const int r = blockIdx.x, s = r / g.rps, j = r - s * g.rps;
    const RowDesc rd = row_desc(kind, d, s, j, aux);
    if (threadIdx.x == 0) {
        d.row_pos[r] = rd.active ? rd.pos : -1;
        d.row_tok[r] = rd.tok;
        if (j == 0) {
            int n = 0;
            for (int jj = 0; jj < g.rps; ++jj) n += row_desc(kind, d, s, jj, aux).active;
            d.n_rows[s] = n;
        }
    }
    if (!rd.active) return;
    const int dm = m.cfg.d_model;
    float *xrow = d.xres + (size_t)r * dm;
    if (kind == KIND_MB) {
        const float *h = d.hpend + ((size_t)s * (d.block_b + 1) + j) * dm;
        const int e = rd.tok;
        for (int i = threadIdx.x; i < dm; i += blockDim.x) {
            float v = h[i];
            if (e > 0 && d.use_posemb) v += __bfloat162float(m.posemb[(size_t)(e - 1) * dm + i]);
            xrow[i] = v;
        }
    } else if (kind == KIND_PREFILL_B) {
        const float *h = d.hidden + (size_t)r * dm;
        for (int i = threadIdx.x; i < dm; i += blockDim.x) xrow[i] = h[i];
    } else {
        const bf16 *e = m.embed + (size_t)rd.tok * dm;
        for (int i = threadIdx.x; i < dm; i += blockDim.x) xrow[i] = __bfloat162float(e[i]);
    }
    __syncthreads();
    rmsnorm_row(xrow, m.norm1, dm, m.cfg.rms_eps, r, g.nt, d.xn, nullptr, red);
}

// x += sum of the split-K partials of the projection that just ran; then RMSNorm.
__global__ void __launch_bounds__(ROW_THREADS) k_add_norm(DevPtrs d, Geom g, int dm, float eps, const bf16 *gain,
                                                          int S, int write_hidden) {
    __shared__ float red[33];
    const int r = blockIdx.x;
    if (d.row_pos[r] < 0) return;
    float *xrow = d.xres + (size_t)r * dm;
    const size_t sstride = (size_t)g.nt * 8 * dm;
    const float *p = d.part + (size_t)r * dm;
    for (int i = threadIdx.x; i < dm; i += blockDim.x) {
        float v = xrow[i];
        for (int s = 0; s < S; ++s) v += p[s * sstride + i];
        xrow[i] = v;
    }
    __syncthreads();
    rmsnorm_row(xrow, gain, dm, eps, r, g.nt, d.xn, write_hidden ? d.hidden + (size_t)r * dm : nullptr, red);
}

// Sums the QKV partials, rotates q and k (rotate-half pairs (i, i + hd/2)) at the
// row's absolute position, stores q as fp32 and appends k, v to the bf16 cache.
__global__ void __launch_bounds__(ROW_THREADS) k_rope_append(DevPtrs d, ModelDev m, Geom g, int layer, int S) {
    const int r = blockIdx.x;
    const int pos = d.row_pos[r];
    if (pos < 0) return;
    const int s = r / g.rps;
    const int H = m.cfg.n_heads, Hkv = m.cfg.n_kv_heads, hd = m.hd, half = hd >> 1, qrows = m.qrows;
    const size_t sstride = (size_t)g.nt * 8 * qrows;
    const float *p = d.part + (size_t)r * qrows;
    auto val = [&](int idx) { float v = 0.f; for (int ss = 0; ss < S; ++ss) v += p[ss * sstride + idx]; return v; };
    const float2 *cs = m.rope + (size_t)pos * half;
    // q and k heads: one thread per rotation pair
    const int n_pairs = (H + Hkv) * half;
    for (int i = threadIdx.x; i < n_pairs; i += blockDim.x) {
        const int head = i / half, ii = i - head * half;
        const float a = val(head * hd + ii), b = val(head * hd + ii + half);
        const float2 c = cs[ii];
        const float ra = a * c.x - b * c.y, rb = b * c.x + a * c.y;
        if (head < H) {
            float *q = d.q + (size_t)r * H * hd + head * hd;
            q[ii] = ra; q[ii + half] = rb;
        } else {
            const int kh = head - H;
            bf16 *kc = m.kcache + ((((size_t)layer * d.max_batch + s) * Hkv + kh) * d.max_ctx + pos) * hd;
            kc[ii] = __float2bfloat16(ra); kc[ii + half] = __float2bfloat16(rb);
        }
    }
    for (int i = threadIdx.x; i < Hkv * hd; i += blockDim.x) {
        const int kh = i / hd, ii = i - kh * hd;
        bf16 *vc = m.vcache + ((((size_t)layer * d.max_batch + s) * Hkv + kh) * d.max_ctx + pos) * hd;
        vc[ii] = __float2bfloat16(val((H + Hkv) * hd + i));
    }
}

// act = silu(gate) * up from the partials of the fused gate/up projection
// (columns [0,F) gate, [F,2F) up), as bf16 in fragment order for the down projection.
__global__ void __launch_bounds__(ROW_THREADS) k_swiglu(DevPtrs d, Geom g, int F, int S) {
    const int r = blockIdx.y;
    if (d.row_pos[r] < 0) return;
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= F) return;
    const size_t sstride = (size_t)g.nt * 8 * 2 * F;
    const float *p = d.part + (size_t)r * 2 * F;
    float gt = 0.f, up = 0.f;
    for (int s = 0; s < S; ++s) { gt += p[s * sstride + f]; up += p[s * sstride + F + f]; }
    const float a = gt / (1.f + expf(-gt)) * up;
    d.act[xfrag_index(r, f, g.nt)] = __float2bfloat16(a);
}
