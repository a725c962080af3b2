// Phases of the forward kernel other than the streams themselves: row set-up,
// input rows, and the per-tile epilogues of the projections (which also prepare
// the input of the projection that follows).
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
            // a draft step beyond the window, or before the queued hidden rows were scored, is a no-op
            if (st.gamma >= st.gamma_max || (!st.sched && st.gamma - st.k_round * d.block_b >= d.block_b)) break;
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
            if (st.gamma - st.k_round * d.block_b < d.block_b) break;     // no whole block is waiting: a no-op
            if (j < st.n_pend) { r.active = 1; r.pos = st.len_B + j; r.tok = d.hpend_e[s * (d.block_b + 1) + j]; }
            break;
        }
    }
    return r;
}

// ------------------------------------------------------------------ input rows

// x = embedding row (or h + e for the pre-verification model, or the draft's
// hidden row during its prefill), spread over the MMA warps of the grid by
// 16-column tiles.  Leaves x (fp32), x * gain of the first RMSNorm (split bf16,
// operand order) and the per-tile sums of squares.
__device__ __forceinline__ void phase_begin(Ctx &c, const Args &a) {
    const DevPtrs &d = a.d;
    const ModelDev &m = a.m;
    const XLay xl{a.g.nt, a.g.G};
    const int dm = m.cfg.d_model, ntiles = dm >> 4, rpad = a.g.rpad;
    const int half = c.lane >> 4, col16 = c.lane & 15;
    for (int tile = c.cta * MMA_WARPS + c.warp; tile < ntiles; tile += c.ncta * MMA_WARPS) {
        const int col = tile * 16 + col16;
        const float gain = __bfloat162float(m.norm1[col]);
        for (int rc = 0; rc < rpad; rc += 32) {             // 32 rows at a time
            float vv[16];                                   // their loads in flight together (the phase is a latency chain)
#pragma unroll
            for (int it = 0; it < 16; ++it) {
                const int r = rc + 2 * it + half;
                float v = 0.f;
                if (rc + 2 * it < rpad && r < a.g.rtot && c.row_pos[r] >= 0) {
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
                }
                vv[it] = v;
            }
#pragma unroll
            for (int it = 0; it < 16; ++it) {
                if (rc + 2 * it >= rpad) break;
                const int r = rc + 2 * it + half;
                const float v = vv[it];
                d.xres[(size_t)r * dm + col] = v;          // idle rows hold zeros: they stay finite through the layers
                store_split(a.fb.xg, xl, r, col, v * gain);
                float ss = v * v;
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
                if (col16 == 0) a.fb.ssq[tile * MAX_ROWS + r] = ss;
            }
        }
    }
}

// ------------------------------------------------------------------ tile epilogues
// acc element (nt, i): token row nt*8 + 2t + (i & 1), tile column g + 8*(i >> 1), with g = lane / 4, t = lane % 4.

// q/k/v tile: the deferred 1/rms of the input RMSNorm, then qkv[k slice][row][column] (the attention phase
// adds the k slices' shares when it reads the rows).
template <int NT>
__device__ __forceinline__ void epi_qkv(Ctx &c, const Args &a, int slice, int tile, int rb, float (&acc)[NT][4]) {
    const int g = c.lane >> 2, t = c.lane & 3, N = a.m.qrows;
    const int n0 = tile * 16 + g, n1 = n0 + 8;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int r0 = rb + nt * 8 + 2 * t;
        const float i0 = c.inv_rms[r0], i1 = c.inv_rms[r0 + 1];
        float *q0 = a.fb.qkv + ((size_t)slice * MAX_ROWS + r0) * N, *q1 = q0 + N;
        if (n0 < N) { q0[n0] = acc[nt][0] * i0; q1[n0] = acc[nt][1] * i1; }
        if (n1 < N) { q0[n1] = acc[nt][2] * i0; q1[n1] = acc[nt][3] * i1; }
    }
}

// Tile of the attention-output / down projection.  The accumulators started from
// the residual rows, so they hold the new x: store it, store x * gain of the
// RMSNorm that follows as split bf16 in operand order (the next projection's input),
// and the tile's share of sum(x^2) per row.
template <int NT>
__device__ __forceinline__ void epi_residual(Ctx &c, const Args &a, const bf16 *gain_next, int tile, int rb, float (&acc)[NT][4]) {
    const int g = c.lane >> 2, t = c.lane & 3, dm = a.m.cfg.d_model;
    const XLay xl{NT, NT <= 4 ? 1 : a.g.G};    // (at most 32 rows: one group, known at compile time)
    const int n0 = tile * 16 + g, n1 = n0 + 8;
    const float g0 = n0 < dm ? __bfloat162float(gain_next[n0]) : 0.f, g1 = n1 < dm ? __bfloat162float(gain_next[n1]) : 0.f;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        float ss[2] = {0.f, 0.f};
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int r = rb + nt * 8 + 2 * t + i;
            float *x = a.d.xres + (size_t)r * dm;
            if (n0 < dm) {
                const float v = acc[nt][i];
                x[n0] = v; ss[i] += v * v;
                store_split(a.fb.xg, xl, r, n0, v * g0);
            }
            if (n1 < dm) {
                const float v = acc[nt][2 + i];
                x[n1] = v; ss[i] += v * v;
                store_split(a.fb.xg, xl, r, n1, v * g1);
            }
        }
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
            ss[0] += __shfl_xor_sync(0xffffffffu, ss[0], o);
            ss[1] += __shfl_xor_sync(0xffffffffu, ss[1], o);
        }
        if (g == 0) {
            a.fb.ssq[tile * MAX_ROWS + rb + nt * 8 + 2 * t] = ss[0];
            a.fb.ssq[tile * MAX_ROWS + rb + nt * 8 + 2 * t + 1] = ss[1];
        }
    }
}

// One k slice of a residual-projection tile: stored as a partial, nothing waits for it.
template <int NT>
__device__ __forceinline__ void epi_partial(Ctx &c, const Args &a, const GemmOp &op, int slice, int tile, int rb, float (&acc)[NT][4]) {
    const int g = c.lane >> 2, t = c.lane & 3;
    float *mine = a.fb.part + ((size_t)slice * op.MT + tile) * (a.g.rpad * 16);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int r0 = rb + nt * 8 + 2 * t;
        mine[r0 * 16 + g] = acc[nt][0];
        mine[(r0 + 1) * 16 + g] = acc[nt][1];
        mine[r0 * 16 + g + 8] = acc[nt][2];
        mine[(r0 + 1) * 16 + g + 8] = acc[nt][3];
    }
}

// After the grid barrier that completes the partials of a k-sliced residual
// projection: x += the slices' sums (slice order, so the result does not depend
// on timing); x * gain of the next RMSNorm as split bf16; sum(x^2) per tile.
// Spread over the MMA warps of the grid by 16-column tiles.
template <int NT, bool BIG>
__device__ __forceinline__ void phase_residual(Ctx &c, const Args &a, const GemmOp &op, const bf16 *gain_next) {
    const XLay xl{NT, NT <= 4 ? 1 : a.g.G};    // (at most 32 rows: one group, known at compile time)
    // A task is one 16-column tile x RT rows: a warp's loads (rows x slices) all fly together and must fit its
    // registers (up to 24 rows they do at once; beyond, 16 rows per task also give every warp of the grid work).
    constexpr int RT = (NT <= 3 && !BIG) ? NT * 8 : 16, NIT = RT / 2;
    const int dm = a.m.cfg.d_model, ntiles = dm >> 4, rpad = BIG ? a.g.rpad : NT * 8, nrc = (rpad + RT - 1) / RT;
    const int half = c.lane >> 4, col16 = c.lane & 15;
    for (int task = c.cta * MMA_WARPS + c.warp; task < ntiles * nrc; task += c.ncta * MMA_WARPS) {
        const int tile = task / nrc, rc = (task - tile * nrc) * RT;
        const int col = tile * 16 + col16;
        const float gain = __bfloat162float(gain_next[col]);
        float v[NIT];
#pragma unroll
        for (int it = 0; it < NIT; ++it)
            v[it] = rc + 2 * it < rpad ? __ldcg(a.d.xres + (size_t)(rc + 2 * it + half) * dm + col) : 0.f;
        for (int s0 = 0; s0 < op.S; s0 += 4) {          // four slices' loads in flight together
            float p[4][NIT];
#pragma unroll
            for (int ds = 0; ds < 4; ++ds)
#pragma unroll
                for (int it = 0; it < NIT; ++it)
                    p[ds][it] = (s0 + ds < op.S && rc + 2 * it < rpad)
                        ? __ldcg(a.fb.part + (((size_t)(s0 + ds) * op.MT + tile) * rpad + rc + 2 * it + half) * 16 + col16) : 0.f;
#pragma unroll
            for (int ds = 0; ds < 4; ++ds)              // slice order: the sum does not depend on timing
#pragma unroll
                for (int it = 0; it < NIT; ++it) v[it] += p[ds][it];
        }
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            if (rc + 2 * it >= rpad) break;
            const int r = rc + 2 * it + half;
            a.d.xres[(size_t)r * dm + col] = v[it];
            store_split(a.fb.xg, xl, r, col, v[it] * gain);
            float ss = v[it] * v[it];
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
            if (col16 == 0) a.fb.ssq[tile * MAX_ROWS + r] = ss;
        }
    }
}

// Interleaved gate/up tile: rows 0..7 are gate rows f = 8*tile + g, rows 8..15 the
// up rows of the same f, so a lane holds both; 1/rms of the input RMSNorm, then
// silu(gate) * up as split bf16 in the operand order the down projection reads.
template <int NT>
__device__ __forceinline__ void epi_swiglu(Ctx &c, const Args &a, int tile, int rb, float (&acc)[NT][4]) {
    const int g = c.lane >> 2, t = c.lane & 3, F = a.m.cfg.d_ffn;
    const XLay xl{NT, NT <= 4 ? 1 : a.g.G};    // (at most 32 rows: one group, known at compile time)
    const int f = tile * 8 + g;
    if (f >= F) return;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int r = rb + nt * 8 + 2 * t + i;
            const float inv = c.inv_rms[r];
            const float gt = acc[nt][i] * inv, up = acc[nt][2 + i] * inv;
            const float v = (r < a.g.rtot && c.row_pos[r] >= 0) ? gt / (1.f + expf(-gt)) * up : 0.f;
            store_split(a.d.act, xl, r, f, v);
        }
    }
}

// LM-head tile: 1/rms of the final RMSNorm, planted bias, logits to their
// destination rows, and the tile's (max, argmax, runner-up) per row.
template <int NT>
__device__ __forceinline__ void epi_head(Ctx &c, const Args &a, float *const *row_dst, const int *bias_at, int tile, int rb,
                                         float (&acc)[NT][4]) {
    const int g = c.lane >> 2, t = c.lane & 3, V = a.m.cfg.vocab;
    const int n0 = tile * 16 + g, n1 = n0 + 8;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int r = rb + nt * 8 + 2 * t + i;
            float *dst = row_dst[r];
            Top2 tp{-INFINITY, 0x7fffffff, -INFINITY};
            if (dst) {
                const int b = bias_at[r];
                const float inv = c.inv_rms[r];
                if (n0 < V) {
                    const float v = acc[nt][i] * inv + (n0 == b ? a.d.succ_bias : 0.f);
                    dst[n0] = v;
                    tp.v1 = v; tp.i1 = n0;
                }
                if (n1 < V) {
                    const float v = acc[nt][2 + i] * inv + (n1 == b ? a.d.succ_bias : 0.f);
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

// Top-2 over the eight MMA warps; every thread gets the result.  sm: 8 entries.
__device__ __forceinline__ Top2 mma_block_top2(Top2 t, Top2 *sm) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Top2 u;
        u.v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
        u.i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
        u.v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
        t = top2_merge(t, u);
    }
    bsync();
    if (lane == 0) sm[w] = t;
    bsync();
    Top2 r = sm[0];
#pragma unroll
    for (int i = 1; i < MMA_WARPS; ++i) r = top2_merge(r, sm[i]);
    return r;
}

// Sum over the eight MMA warps; every thread gets the result.  red: 8 floats.
__device__ __forceinline__ float mma_block_sum(float v, float *red) {
    v = warp_sum(v);
    bsync();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    bsync();
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < MMA_WARPS; ++i) s += red[i];
    return s;
}

// Arg-max (lowest index on ties) and gap to the runner-up of LM-head row r from
// the per-tile results; the MMA warps of the block work on one row.
__device__ __forceinline__ void head_row_argmax(const Args &a, int r, Top2 *sm) {
    const int MT = a.P.op[OP_HEAD].MT;
    Top2 t{-INFINITY, 0x7fffffff, -INFINITY};
    for (int tile = threadIdx.x; tile < MT; tile += MMA_THREADS) {
        const float4 v = __ldcg(reinterpret_cast<const float4 *>(a.fb.tile_top) + (size_t)tile * MAX_ROWS + r);
        t = top2_merge(t, Top2{v.x, __float_as_int(v.y), v.z});
    }
    t = mma_block_top2(t, sm);
    if (threadIdx.x == 0) { a.d.row_arg[r] = t.i1; a.d.row_margin[r] = t.v1 - t.v2; }
    bsync();
}

}  // namespace fwd
