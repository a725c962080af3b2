// Weight stream of the forward kernel: the static list of weight units of one
// warp, the bulk-copy producer that walks it, and the projection loop that
// consumes it with tensor cores.
#pragma once
#include "forward.cuh"

namespace fwd {

// Position in the static unit list of (block, warp): projection q (layer-major:
// 4 per layer, then the LM head), item ordinal m of this block, tile ordinal j of
// this warp, unit ordinal u inside the k slice.
struct Cursor {
    int q, m, j, u;
    int done;
    // derived by settle()
    int opi, layer, tile, k, kc;
};

__device__ __forceinline__ int first_item(const GemmOp &op, int cta, int ncta) {
    int f = cta - op.rot;
    return f < 0 ? f + ncta : f;
}

// Moves the cursor to the next existing unit at or after its position.
__device__ __forceinline__ bool settle(Cursor &cu, const Plan &P, int cta, int ncta, int warp) {
    const int nq = 4 * P.n_layers + (P.has_head ? 1 : 0);
    while (true) {
        if (cu.q >= nq) { cu.done = 1; return false; }
        const int opi = cu.q < 4 * P.n_layers ? (cu.q & 3) : OP_HEAD;
        const GemmOp &op = P.op[opi];
        const int idx = first_item(op, cta, ncta) + cu.m * ncta;
        if (idx >= op.items) { ++cu.q; cu.m = cu.j = cu.u = 0; continue; }
        const int s = idx % op.S, g = idx / op.S;
        const int t_lo = g * op.TPG, t_hi = min(op.MT, t_lo + op.TPG);
        const int tile = t_lo + warp + MMA_WARPS * cu.j;
        if (tile >= t_hi) { ++cu.m; cu.j = cu.u = 0; continue; }
        const int k_lo = s * op.KS, k_hi = min(op.K, k_lo + op.KS);
        const int k = k_lo + cu.u * KC;
        if (k >= k_hi) { ++cu.j; cu.u = 0; continue; }
        cu.opi = opi;
        cu.layer = cu.q < 4 * P.n_layers ? (cu.q >> 2) : 0;
        cu.tile = tile;
        cu.k = k;
        cu.kc = min(KC, k_hi - k);
        return true;
    }
}

struct Stream {
    Cursor cu;
    int pn, cn;            // units issued / consumed by this warp
};

// Issues the bulk copies of the cursor's unit into the next stage and advances the cursor.
__device__ __forceinline__ void issue_unit(Ctx &c, Stream &st, const Plan &P) {
    if (st.cu.done) return;
    const int slot = st.pn % STAGES;
    unsigned char *stage = c.ring + slot * STAGE_BYTES;
    uint64_t *bar = c.mbar + slot;
    const GemmOp &op = P.op[st.cu.opi];
    const uint32_t bytes = (uint32_t)st.cu.kc * 2u;
    if (c.lane == 0) mbar_expect_tx(bar, 16u * bytes);
    __syncwarp();
    if (c.lane < 16) {
        const bf16 *src;
        if (op.interleave) {
            const int F = op.N >> 1;
            const int f = min(st.cu.tile * 8 + (c.lane & 7), F - 1);
            src = (c.lane < 8 ? op.W1 : op.W2) + (size_t)st.cu.layer * op.lstride + (size_t)f * op.K + st.cu.k;
        } else {
            const int n = min(st.cu.tile * 16 + c.lane, op.N - 1);
            src = op.W1 + (size_t)st.cu.layer * op.lstride + (size_t)n * op.K + st.cu.k;
        }
        bulk_g2s(stage + c.lane * PITCH, src, bytes, bar, c.policy);
    }
    ++st.pn;
    ++st.cu.u;
    settle(st.cu, P, c.cta, c.ncta, c.warp);
}

// Bounded wait on a shared-memory barrier phase.
__device__ __forceinline__ void wait_bar(Ctx &c, const FwdBufs &fb, uint64_t *bar, uint32_t parity, int code) {
    unsigned it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if (++it > SPIN_LIMIT) {
            if (c.lane == 0) atomicExch(fb.abort_flag, code);
            break;
        }
    }
}

// Bounded wait for the stage that holds unit number n of this warp.
__device__ __forceinline__ void wait_unit(Ctx &c, const FwdBufs &fb, int n) {
    wait_bar(c, fb, c.mbar + (n % STAGES), (uint32_t)(n / STAGES) & 1u, 2);
}

// Streaming warp -> its epilogue partner: the accumulators of a finished tile,
// through shared memory in lane order (conflict free), one tile at a time.
template <int NT>
__device__ __forceinline__ void hand_over(Ctx &c, const FwdBufs &fb, const float (&acc)[NT][4]) {
    wait_bar(c, fb, c.hand_empty, ((uint32_t)c.n_hand & 1u) ^ 1u, 3);      // the partner took the previous tile
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) c.hand[(nt * 4 + i) * 32 + c.lane] = acc[nt][i];
    __syncwarp();
    if (c.lane == 0) mbar_arrive(c.hand_full);
    ++c.n_hand;
}
template <int NT>
__device__ __forceinline__ void receive(Ctx &c, const FwdBufs &fb, float (&acc)[NT][4]) {
    wait_bar(c, fb, c.hand_full, (uint32_t)c.n_hand & 1u, 4);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nt][i] = c.hand[(nt * 4 + i) * 32 + c.lane];
    __syncwarp();
    if (c.lane == 0) mbar_arrive(c.hand_empty);
    ++c.n_hand;
}

// acc[nt] += W(16 rows x 32*nchunks k) * X over one stage.  Lane (g, t) reads the
// 8 consecutive weights of rows g and g+8 at k = 32c + 8t and uses them as the k
// slots {2t, 2t+1, 2t+8, 2t+9} of two MMAs; the activation fragments are stored
// with the same rule, so the products pair up.
template <int NT>
__device__ __forceinline__ void consume_unit(const unsigned char *stage, const uint4 *xs, int chunk0, int nchunks,
                                             float (&acc)[NT][4], int lane) {
    const int g = lane >> 2, t = lane & 3;
    const unsigned char *p0 = stage + g * PITCH + t * 16, *p1 = p0 + 8 * PITCH;
#pragma unroll 2
    for (int cix = 0; cix < nchunks; ++cix) {
        const uint4 a0 = *reinterpret_cast<const uint4 *>(p0 + cix * 64);
        const uint4 a1 = *reinterpret_cast<const uint4 *>(p1 + cix * 64);
        const uint4 *xb = xs + (size_t)(chunk0 + cix) * (NT * 32) + lane;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const uint4 b = xb[nt * 32];
            mma16816(acc[nt], a0.x, a1.x, a0.y, a1.y, b.x, b.y);
            mma16816(acc[nt], a0.z, a1.z, a0.w, a1.w, b.z, b.w);
        }
    }
}

// Split-k reduction of one 16-column tile.  The warp stores its slice's partial,
// counts itself in, and the warp that arrives last adds the slices up in slice
// order.  Returns true for that warp, with the complete sums in acc.
// Accumulator element (nt, i): token row nt*8 + 2t + (i & 1), tile column g + 8*(i >> 1).
template <int NT>
__device__ __forceinline__ bool tile_reduce(Ctx &c, const FwdBufs &fb, const GemmOp &op, int tile, int s,
                                            float (&acc)[NT][4]) {
    if (op.S == 1) return true;
    constexpr int RPAD = NT * 8;
    const int g = c.lane >> 2, t = c.lane & 3;
    float *mine = fb.part + ((size_t)s * op.MT + tile) * (RPAD * 16);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int r0 = nt * 8 + 2 * t;
        mine[r0 * 16 + g] = acc[nt][0];
        mine[(r0 + 1) * 16 + g] = acc[nt][1];
        mine[r0 * 16 + g + 8] = acc[nt][2];
        mine[(r0 + 1) * 16 + g + 8] = acc[nt][3];
    }
    __threadfence();
    __syncwarp();
    int old = 0;
    if (c.lane == 0) old = atomicAdd(fb.tile_cnt + tile, 1);
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old != op.S - 1) return false;
    if (c.lane == 0) fb.tile_cnt[tile] = 0;        // the next projection starts from zero (a grid barrier lies between)
    __threadfence();
    float sum[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) sum[nt][0] = sum[nt][1] = sum[nt][2] = sum[nt][3] = 0.f;
    for (int ss = 0; ss < op.S; ++ss) {
        if (ss == s) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) sum[nt][i] += acc[nt][i];
        } else {
            const float *p = fb.part + ((size_t)ss * op.MT + tile) * (RPAD * 16);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int r0 = nt * 8 + 2 * t;
                sum[nt][0] += __ldcg(p + r0 * 16 + g);
                sum[nt][1] += __ldcg(p + (r0 + 1) * 16 + g);
                sum[nt][2] += __ldcg(p + r0 * 16 + g + 8);
                sum[nt][3] += __ldcg(p + (r0 + 1) * 16 + g + 8);
            }
        }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nt][i] = sum[nt][i];
    return true;
}

// One projection: for every item of this block load the activation slice, then
// every streaming warp runs its tiles through its pipeline and hands each
// finished tile to its partner.  xload(k_lo, k_hi) fills the scratch with the
// slice in fragment order (all threads call it); epi(tile, acc) runs in the
// epilogue warp that completed the tile (last k slice to arrive).
template <int NT, class XLoad, class Epi>
__device__ __forceinline__ void gemm_op(Ctx &c, const FwdBufs &fb, const Plan &P, int opi, Stream &st, XLoad xload,
                                        Epi epi) {
    const GemmOp &op = P.op[opi];
    const uint4 *xs = reinterpret_cast<const uint4 *>(c.scratch);
    const bool streamer = c.warp < MMA_WARPS;
    const int w = c.warp & (MMA_WARPS - 1);
    for (int idx = first_item(op, c.cta, c.ncta); idx < op.items; idx += c.ncta) {
        const int s = idx % op.S, g = idx / op.S;
        const int k_lo = s * op.KS, k_hi = min(op.K, k_lo + op.KS);
        const int t_lo = g * op.TPG, t_hi = min(op.MT, t_lo + op.TPG);
        __syncthreads();                       // the scratch is free
        xload(k_lo, k_hi);
        __syncthreads();
        for (int tile = t_lo + w; tile < t_hi; tile += MMA_WARPS) {
            float acc[NT][4];
            if (streamer) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
                for (int k = k_lo; k < k_hi; k += KC) {
                    const int kc = min(KC, k_hi - k);
                    wait_unit(c, fb, st.cn);
                    consume_unit<NT>(c.ring + (st.cn % STAGES) * STAGE_BYTES, xs, (k - k_lo) >> 5, kc >> 5, acc, c.lane);
                    ++st.cn;
                    __syncwarp();
                    fence_proxy_async();
                    issue_unit(c, st, P);      // refill the freed stage with the next unit of the static list
                }
                hand_over<NT>(c, fb, acc);
            } else {
                receive<NT>(c, fb, acc);
                if (tile_reduce<NT>(c, fb, op, tile, s, acc)) epi(tile, acc);
            }
        }
    }
}

}  // namespace fwd
