// Phases of the forward kernel other than the weight stream itself: row set-up,
// input rows, activation-slice loaders (with RMSNorm applied on the fly),
// per-tile epilogues of the projections, and the tails that take the loop's
// decisions (Eq. 6 / Eq. 7 / Algorithm 1) on the device.
#pragma once
#include "control.cuh"
#include "fwd_stream.cuh"

namespace fwd {

struct Args {
    DevPtrs d;
    ModelDev m;
    Geom g;
    Plan P;
    FwdBufs fb;
    int32_t kind, aux;
};

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
                const int n_in = st.P - st.len_D;            // 1, or 2 after a fully accepted step
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
            const int p = aux + j;
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

// ------------------------------------------------------------------ input rows

// x = embedding row (or h + e for the pre-verification model, or the draft's
// hidden row during its prefill), spread over all warps of the grid by 16-column
// tiles; also the per-tile sums of squares the first RMSNorm needs.
__device__ __forceinline__ void phase_begin(Ctx &c, const Args &a, int rpad) {
    const DevPtrs &d = a.d;
    const ModelDev &m = a.m;
    const int dm = m.cfg.d_model, ntiles = dm >> 4;
    const int half = c.lane >> 4, col16 = c.lane & 15;
    for (int tile = c.cta * WARPS + c.warp; tile < ntiles; tile += c.ncta * WARPS) {
        const int col = tile * 16 + col16;
        for (int rr = 0; rr < rpad; rr += 2) {
            const int r = rr + half;
            float v = 0.f;
            const bool act = r < a.g.rtot && c.row_pos[r] >= 0;
            if (act) {
                const int s = r / a.g.rps, j = r - s * a.g.rps;
                if (a.kind == KIND_MB) {
                    v = d.hpend[((size_t)s * (d.block_b + 1) + j) * dm + col];
                    const int e = c.row_tok[r];
                    if (e > 0 && d.use_posemb) v += __bfloat162float(m.posemb[(size_t)(e - 1) * dm + col]);
                } else if (a.kind == KIND_PREFILL_B) {
                    v = __ldcg(d.hidden + (size_t)r * dm + col);
                } else {
                    v = __bfloat162float(m.embed[(size_t)c.row_tok[r] * dm + col]);
                }
                d.xres[(size_t)r * dm + col] = v;
            }
            float ss = v * v;
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
            if (col16 == 0 && r < MAX_ROWS) a.fb.ssq[tile * MAX_ROWS + r] = ss;
        }
    }
}

// inv_rms[r] = 1 / sqrt(mean(x_r^2) + eps) from the per-tile sums, in a fixed order.
__device__ __forceinline__ void compute_inv(Ctx &c, const Args &a) {
    const int dm = a.m.cfg.d_model, ntiles = dm >> 4;
    const int r = threadIdx.x >> 3, sub = threadIdx.x & 7;
    float s = 0.f;
    if (r < MAX_ROWS)
        for (int t = sub; t < ntiles; t += 8) s += __ldcg(a.fb.ssq + t * MAX_ROWS + r);
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    s += __shfl_xor_sync(0xffffffffu, s, 4);
    __syncthreads();                            // earlier readers of inv_rms are done
    if (sub == 0 && r < MAX_ROWS) c.inv_rms[r] = rsqrtf(s / (float)dm + a.m.cfg.rms_eps);
    __syncthreads();
}

// ------------------------------------------------------------------ activation slices

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Slice [k_lo, k_hi) of RMSNorm(x) * gain as bf16 in fragment order:
// [chunk of 32 k][row tile][lane = (r % 8) * 4 + (k % 32) / 8] x 8 values.
template <int NT>
__device__ __forceinline__ void xload_normed(Ctx &c, const Args &a, const bf16 *gain, int k_lo, int k_hi) {
    uint4 *xs = reinterpret_cast<uint4 *>(c.scratch);
    const int dm = a.m.cfg.d_model;
    const int npieces = (k_hi - k_lo) >> 3;
    for (int i = threadIdx.x; i < NT * 8 * npieces; i += THREADS) {
        const int r = i / npieces, p = i - r * npieces, k = k_lo + p * 8;
        uint4 out = make_uint4(0u, 0u, 0u, 0u);
        if (r < a.g.rtot && c.row_pos[r] >= 0) {
            const float4 x0 = __ldcg(reinterpret_cast<const float4 *>(a.d.xres + (size_t)r * dm + k));
            const float4 x1 = __ldcg(reinterpret_cast<const float4 *>(a.d.xres + (size_t)r * dm + k + 4));
            const uint4 gw = *reinterpret_cast<const uint4 *>(gain + k);
            const __nv_bfloat162 *g2 = reinterpret_cast<const __nv_bfloat162 *>(&gw);
            const float inv = c.inv_rms[r];
            const float2 ga = __bfloat1622float2(g2[0]), gb = __bfloat1622float2(g2[1]);
            const float2 gc = __bfloat1622float2(g2[2]), gd = __bfloat1622float2(g2[3]);
            out.x = pack_bf16x2(x0.x * inv * ga.x, x0.y * inv * ga.y);
            out.y = pack_bf16x2(x0.z * inv * gb.x, x0.w * inv * gb.y);
            out.z = pack_bf16x2(x1.x * inv * gc.x, x1.y * inv * gc.y);
            out.w = pack_bf16x2(x1.z * inv * gd.x, x1.w * inv * gd.y);
        }
        xs[((p >> 2) * NT + (r >> 3)) * 32 + ((r & 7) << 2) + (p & 3)] = out;
    }
}

// Slice of a bf16 buffer that already is in fragment order in global memory.
template <int NT>
__device__ __forceinline__ void xload_frag(Ctx &c, const bf16 *src, int k_lo, int k_hi) {
    uint4 *xs = reinterpret_cast<uint4 *>(c.scratch);
    const uint4 *s4 = reinterpret_cast<const uint4 *>(src) + (size_t)(k_lo >> 5) * (NT * 32);
    const int n = ((k_hi - k_lo) >> 5) * (NT * 32);
    for (int i = threadIdx.x; i < n; i += THREADS) xs[i] = __ldcg(s4 + i);
}

// ------------------------------------------------------------------ tile epilogues

// Complete q/k/v sums of a tile -> qkv[row][column].
template <int NT>
__device__ __forceinline__ void epi_qkv(Ctx &c, const Args &a, int tile, float (&acc)[NT][4]) {
    const int g = c.lane >> 2, t = c.lane & 3, N = a.m.qrows;
    const int n0 = tile * 16 + g, n1 = n0 + 8;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int r0 = nt * 8 + 2 * t;
        float *q0 = a.fb.qkv + (size_t)r0 * N, *q1 = q0 + N;
        if (n0 < N) { q0[n0] = acc[nt][0]; q1[n0] = acc[nt][1]; }
        if (n1 < N) { q0[n1] = acc[nt][2]; q1[n1] = acc[nt][3]; }
    }
}

// Residual add of a tile of the attention-output / down projection, and the
// tile's share of sum(x^2) per row for the RMSNorm that follows.
template <int NT>
__device__ __forceinline__ void epi_residual(Ctx &c, const Args &a, int tile, float (&acc)[NT][4]) {
    const int g = c.lane >> 2, t = c.lane & 3, dm = a.m.cfg.d_model;
    const int n0 = tile * 16 + g, n1 = n0 + 8;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        float ss[2] = {0.f, 0.f};
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int r = nt * 8 + 2 * t + i;
            if (r < a.g.rtot && c.row_pos[r] >= 0) {
                float *x = a.d.xres + (size_t)r * dm;
                if (n0 < dm) { const float v = __ldcg(x + n0) + acc[nt][i]; x[n0] = v; ss[i] += v * v; }
                if (n1 < dm) { const float v = __ldcg(x + n1) + acc[nt][2 + i]; x[n1] = v; ss[i] += v * v; }
            }
        }
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
            ss[0] += __shfl_xor_sync(0xffffffffu, ss[0], o);
            ss[1] += __shfl_xor_sync(0xffffffffu, ss[1], o);
        }
        if (g == 0) {
            a.fb.ssq[tile * MAX_ROWS + nt * 8 + 2 * t] = ss[0];
            a.fb.ssq[tile * MAX_ROWS + nt * 8 + 2 * t + 1] = ss[1];
        }
    }
}

// Interleaved gate/up tile: rows 0..7 are gate rows f = 8*tile + g, rows 8..15 the
// up rows of the same f, so a lane holds both and writes silu(gate) * up as bf16
// in the fragment order the down projection reads.
template <int NT>
__device__ __forceinline__ void epi_swiglu(Ctx &c, const Args &a, int tile, float (&acc)[NT][4]) {
    const int g = c.lane >> 2, t = c.lane & 3, F = a.m.cfg.d_ffn;
    const int f = tile * 8 + g;
    if (f >= F) return;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int r = nt * 8 + 2 * t + i;
            const float gt = acc[nt][i], up = acc[nt][2 + i];
            const float v = gt / (1.f + expf(-gt)) * up;
            a.d.act[xfrag_index(r, f, NT)] = __float2bfloat16(v);
        }
    }
}

// LM-head tile: logits (+ planted bias) to their destination rows, and the
// tile's (max, argmax, runner-up) per row.
template <int NT>
__device__ __forceinline__ void epi_head(Ctx &c, const Args &a, float *const *row_dst, const int *bias_at, int tile,
                                         float (&acc)[NT][4]) {
    const int g = c.lane >> 2, t = c.lane & 3, V = a.m.cfg.vocab;
    const int n0 = tile * 16 + g, n1 = n0 + 8;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int r = nt * 8 + 2 * t + i;
            float *dst = row_dst[r];
            Top2 tp{-INFINITY, 0x7fffffff, -INFINITY};
            if (dst) {
                const int b = bias_at[r];
                if (n0 < V) {
                    const float v = acc[nt][i] + (n0 == b ? a.d.succ_bias : 0.f);
                    dst[n0] = v;
                    tp.v1 = v; tp.i1 = n0;
                }
                if (n1 < V) {
                    const float v = acc[nt][2 + i] + (n1 == b ? a.d.succ_bias : 0.f);
                    dst[n1] = v;
                    tp = top2_merge(tp, Top2{v, n1, -INFINITY});
                }
            }
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
                Top2 u;
                u.v1 = __shfl_xor_sync(0xffffffffu, tp.v1, o);
                u.i1 = __shfl_xor_sync(0xffffffffu, tp.i1, o);
                u.v2 = __shfl_xor_sync(0xffffffffu, tp.v2, o);
                tp = top2_merge(tp, u);
            }
            if (g == 0 && dst)
                reinterpret_cast<float4 *>(a.fb.tile_top)[(size_t)tile * MAX_ROWS + r] =
                    make_float4(tp.v1, __int_as_float(tp.i1), tp.v2, 0.f);
        }
    }
}

// Arg-max (lowest index on ties) and gap to the runner-up of LM-head row r from
// the per-tile results; the whole block works on one row.
__device__ __forceinline__ void head_row_argmax(const Args &a, int r, Top2 *sm) {
    const int MT = a.P.op[OP_HEAD].MT;
    Top2 t{-INFINITY, 0x7fffffff, -INFINITY};
    for (int tile = threadIdx.x; tile < MT; tile += THREADS) {
        const float4 v = __ldcg(reinterpret_cast<const float4 *>(a.fb.tile_top) + (size_t)tile * MAX_ROWS + r);
        t = top2_merge(t, Top2{v.x, __float_as_int(v.y), v.z});
    }
    __syncthreads();
    t = block_top2(t, sm);
    if (threadIdx.x == 0) { a.d.row_arg[r] = t.i1; a.d.row_margin[r] = t.v1 - t.v2; }
    __syncthreads();
}

}  // namespace fwd
