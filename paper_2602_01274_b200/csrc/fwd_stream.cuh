// Weight and activation streams of the forward kernel: the two producer warps
// and the projection loop of the MMA warps.
//
// Order of everything, identical on both sides: projections q = 0, 1, ... of the
// forward (four per layer, then the LM head); inside a projection the passes of
// this block (at most MAX_TILES tiles each, evenly sized); inside a pass the k steps of KC
// columns; inside a k step the tiles of the pass.  Weight unit number n of the
// block lives in ring stage n % NS, activation chunk number m in stage m % XS.
#pragma once
#include "forward.cuh"

namespace fwd {

// Bounded wait on a shared-memory barrier phase.  Returns false when it gave up
// (its own limit, or another wait of the grid gave up before).
__device__ __forceinline__ bool wait_bar(const FwdBufs &fb, uint64_t *bar, uint32_t parity, int code, int info = 0) {
    unsigned it = 0;
    while (!mbar_try_wait(bar, parity)) {
        ++it;
        if ((it & 1023u) == 0 && (it > MBAR_SPIN_LIMIT || *(volatile int32_t *)fb.abort_flag)) {
            if (atomicCAS(fb.abort_flag, 0, code) == 0) {      // first wait of the grid to give up: leave a note
                fb.abort_flag[1] = blockIdx.x; fb.abort_flag[2] = threadIdx.x >> 5; fb.abort_flag[3] = info;
            }
            return false;
        }
    }
    return true;
}

// Bounded wait until a shared-memory counter written by another warp reaches `want`.
__device__ __forceinline__ void wait_count(const FwdBufs &fb, volatile int32_t *p, int want, int code) {
    unsigned it = 0;
    while (*p < want) {
        ++it;
        if ((it & 1023u) == 0 && (it > SPIN_LIMIT * 4u || *(volatile int32_t *)fb.abort_flag)) {
            if (atomicCAS(fb.abort_flag, 0, code) == 0) {
                fb.abort_flag[1] = blockIdx.x; fb.abort_flag[2] = threadIdx.x >> 5; fb.abort_flag[3] = want;
            }
            break;
        }
    }
}

__device__ __forceinline__ int n_ops(const Plan &P) { return 4 * P.n_layers + (P.has_head ? 1 : 0); }
__device__ __forceinline__ int op_index(const Plan &P, int q) { return q < 4 * P.n_layers ? (q & 3) : OP_HEAD; }
__device__ __forceinline__ int op_layer(const Plan &P, int q) { return q < 4 * P.n_layers ? (q >> 2) : 0; }

// Warps W_PRODUCER ..: every weight unit of the block, for the whole forward, in
// order; producer `me` issues the units n with n % W_PRODUCERS == me.
__device__ __forceinline__ void weight_producer(Ctx &c, const FwdBufs &fb, const Plan &P, int me) {
    int n = 0;
    for (int q = 0; q < n_ops(P); ++q) {
        const GemmOp &op = P.op[op_index(P, q)];
        const size_t lbase = (size_t)op_layer(P, q) * op.lstride;
        int t0, T, k_lo, k_hi;
        op_range(op, c.cta, c.ncta, t0, T, k_lo, k_hi);
        for (int p = 0; p < n_passes(T); ++p) {
            int p0, Tp;
            pass_range(T, p, p0, Tp);
            for (int k = k_lo; k < k_hi; k += KC) {
                const uint32_t bytes = (uint32_t)min(KC, k_hi - k) * 2u;
                for (int i = 0; i < Tp; ++i, ++n) {
                    if (n % W_PRODUCERS != me) continue;
                    const int slot = n % NS, tile = t0 + p0 + i;
                    if (!wait_bar(fb, c.wempty + slot, (((uint32_t)(n / NS)) & 1u) ^ 1u, 5, n)) return;   // stop feeding
                    if (c.lane == 0) mbar_expect_tx(c.wfull + slot, 16u * bytes);
                    __syncwarp();
                    if (c.lane < 16) {
                        const bf16 *src;
                        if (op.interleave) {
                            const int f = min(tile * 8 + (c.lane & 7), (op.N >> 1) - 1);
                            src = (c.lane < 8 ? op.W1 : op.W2) + lbase + (size_t)f * op.K + k;
                        } else {
                            const int nrow = min(tile * 16 + c.lane, op.N - 1);
                            src = op.W1 + lbase + (size_t)nrow * op.K + k;
                        }
                        bulk_g2s(c.ring + slot * STAGE_BYTES + c.lane * PITCH, src, bytes, c.wfull + slot, c.policy);
                    }
                }
            }
        }
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// inv_rms[r] = 1 / sqrt(mean(x_r^2) + eps) from the per-tile sums ssq[tile][row], in a fixed
// order (one warp, lane = row; four running sums keep the loads independent).
__device__ __forceinline__ void compute_inv(Ctx &c, const FwdBufs &fb, int dm, float eps) {
    const int ntiles = dm >> 4;
    const float *p = fb.ssq + c.lane;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    int t = 0;
    for (; t + 4 <= ntiles; t += 4) {
        s0 += __ldcg(p + (t + 0) * MAX_ROWS);
        s1 += __ldcg(p + (t + 1) * MAX_ROWS);
        s2 += __ldcg(p + (t + 2) * MAX_ROWS);
        s3 += __ldcg(p + (t + 3) * MAX_ROWS);
    }
    for (; t < ntiles; ++t) s0 += __ldcg(p + t * MAX_ROWS);
    c.inv_rms[c.lane] = rsqrtf(((s0 + s1) + (s2 + s3)) / (float)dm + eps);
    __syncwarp();
}

// Warps X_PRODUCER .. X_PRODUCER + XS - 1: the activation chunk of every k step,
// once the projection's inputs are complete (the MMA warps raise ready_op[0] after
// the grid barrier): a bulk copy of a bf16 buffer that already has fragment order.
// Stage s is fed by producer s, so its generations stay in order.
template <int NT>
__device__ __forceinline__ void activation_producer(Ctx &c, const FwdBufs &fb, const Plan &P, int me, uint64_t keep_policy) {
    constexpr int XS = x_stages(NT), XSTAGE_BYTES = xstage_bytes(NT);
    if (me >= XS) return;
    int m = 0;
    for (int q = 0; q < n_ops(P); ++q) {
        const GemmOp &op = P.op[op_index(P, q)];
        int t0, T, k_lo, k_hi;
        op_range(op, c.cta, c.ncta, t0, T, k_lo, k_hi);
        if (T == 0) continue;
        wait_count(fb, c.ready_op, q + 1, 6);
        __threadfence_block();
        asm volatile("fence.proxy.async;" ::: "memory");
        for (int p = 0; p < n_passes(T); ++p) {
            for (int k = k_lo; k < k_hi; k += XK, ++m) {
                if (m % XS != me) continue;
                const int slot = m % XS, nch = min(XK, k_hi - k) >> 5;
                if (!wait_bar(fb, c.xempty + slot, (((uint32_t)(m / XS)) & 1u) ^ 1u, 7, m)) return;
                if (c.lane == 0) {                       // the chunk's bf16 values, then its rounding remainders
                    const uint32_t bytes = (uint32_t)nch * (uint32_t)NT * 512u;
                    const bf16 *src = op.X + (size_t)(k >> 5) * NT * 256;
                    unsigned char *dst = c.scratch + slot * XSTAGE_BYTES;
                    mbar_expect_tx(c.xfull + slot, 2u * bytes);
                    bulk_g2s(dst, src, bytes, c.xfull + slot, keep_policy);
                    bulk_g2s(dst + XSTAGE_BYTES / 2, src + op.x_lo, bytes, c.xfull + slot, keep_policy);
                }
                __syncwarp();
            }
        }
    }
}

// Last warp of the block: 1/rms per row for the projections that follow an RMSNorm,
// as soon as the projection's inputs are complete (ready_op[1] tells the epilogues).
__device__ __forceinline__ void helper_warp(Ctx &c, const FwdBufs &fb, const Plan &P, int dm, float eps) {
    for (int q = 0; q < n_ops(P); ++q) {
        const int opi = op_index(P, q);
        if (opi != OP_QKV && opi != OP_GU && opi != OP_HEAD) continue;
        int t0, T, k_lo, k_hi;
        op_range(P.op[opi], c.cta, c.ncta, t0, T, k_lo, k_hi);
        if (T == 0) continue;
        wait_count(fb, c.ready_op, q + 1, 6);
        __threadfence_block();
        compute_inv(c, fb, dm, eps);
        __threadfence_block();
        if (c.lane == 0) c.ready_op[1] = q + 1;
        __syncwarp();
    }
}

// acc[nt] += W(16 rows x 32*nchunks k, from chunk `chunk0` of the stage) * (X_hi + X_lo).  Lane (g, t) reads the
// 8 consecutive weights of rows g and g+8 at k = 32c + 8t and uses them as the k slots {2t, 2t+1, 2t+8, 2t+9}
// of two MMAs; the activation fragments are stored with the same rule, so the products pair up.
template <int NT>
__device__ __forceinline__ void consume_unit(const unsigned char *stage, int chunk0, const uint4 *xhi, const uint4 *xlo, int nchunks,
                                             float (&acc)[NT][4], int lane) {
    const int g = lane >> 2, t = lane & 3;
    const unsigned char *p0 = stage + g * PITCH + t * 16 + chunk0 * 64, *p1 = p0 + 8 * PITCH;
#pragma unroll 2
    for (int cix = 0; cix < nchunks; ++cix) {
        const uint4 a0 = *reinterpret_cast<const uint4 *>(p0 + cix * 64);
        const uint4 a1 = *reinterpret_cast<const uint4 *>(p1 + cix * 64);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const uint4 bh = xhi[(cix * NT + nt) * 32 + lane], bl = xlo[(cix * NT + nt) * 32 + lane];
            mma16816(acc[nt], a0.x, a1.x, a0.y, a1.y, bh.x, bh.y);
            mma16816(acc[nt], a0.z, a1.z, a0.w, a1.w, bh.z, bh.w);
            mma16816(acc[nt], a0.x, a1.x, a0.y, a1.y, bl.x, bl.y);
            mma16816(acc[nt], a0.z, a1.z, a0.w, a1.w, bl.z, bl.w);
        }
    }
}

// One projection, run by the eight MMA warps after the grid barrier that
// completed its inputs.  Warp w owns tile w of every pass, over the block's k
// range; epi(tile, acc) gets the sums.
// Accumulator element (nt, i): token row nt*8 + 2t + (i & 1), tile column g + 8*(i >> 1).
template <int NT, class Epi>
__device__ __forceinline__ void gemm_op(Ctx &c, const FwdBufs &fb, const Plan &P, int q, const float *resid, int resid_ld,
                                        Epi epi) {
    const GemmOp &op = P.op[op_index(P, q)];
    if (threadIdx.x == 0) {
        __threadfence_block();
        c.ready_op[0] = q + 1;                 // the activation producer may start on this projection
    }
    const int opi = op_index(P, q);
    const bool normed = opi == OP_QKV || opi == OP_GU || opi == OP_HEAD;
    int t0, T, k_lo, k_hi;
    op_range(op, c.cta, c.ncta, t0, T, k_lo, k_hi);
    constexpr int XS = x_stages(NT), XSTAGE_BYTES = xstage_bytes(NT);
    for (int p = 0; p < n_passes(T); ++p) {
        int p0, Tp;
        pass_range(T, p, p0, Tp);
        const bool has = c.warp < Tp;
        // Accumulators start from the residual rows when the projection adds into the residual stream: the
        // loads are issued before the k loop, so the epilogue has no global round trip of its own.
        float acc[NT][4];
        {
            const int g = c.lane >> 2, t = c.lane & 3;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[nt][i] = 0.f;
                    if (resid && has) {
                        const int r = nt * 8 + 2 * t + (i & 1), n0 = (t0 + p0 + c.warp) * 16 + g + 8 * (i >> 1);
                        if (n0 < op.N) acc[nt][i] = __ldcg(resid + (size_t)r * resid_ld + n0);
                    }
                }
        }
        for (int k = k_lo; k < k_hi; k += KC) {
            const int nch = min(KC, k_hi - k) >> 5;
            int slot = 0;
            if (has) {
                const int n = c.wn + c.warp;
                slot = n % NS;
                wait_bar(fb, c.wfull + slot, ((uint32_t)(n / NS)) & 1u, 9, n);
            }
            for (int c0 = 0; c0 < nch; c0 += XCH) {           // the activations come in chunks of XK columns
                const int xslot = c.xn % XS;
                wait_bar(fb, c.xfull + xslot, ((uint32_t)(c.xn / XS)) & 1u, 8, c.xn);
                if (has) {
                    const uint4 *xhi = reinterpret_cast<const uint4 *>(c.scratch + xslot * XSTAGE_BYTES);
                    consume_unit<NT>(c.ring + slot * STAGE_BYTES, c0, xhi, xhi + XSTAGE_BYTES / 32, min(XCH, nch - c0), acc, c.lane);
                }
                __syncwarp();
                if (c.lane == 0) mbar_arrive(c.xempty + xslot);
                ++c.xn;
            }
            if (has && c.lane == 0) mbar_arrive(c.wempty + slot);
            // Lockstep over k.  A ring stage is shared by different warps over time, and a parity wait is exact
            // only while the waiter is less than one stage generation ahead: a k step has at most NS units (and
            // at most two activation chunks), so after this barrier the stage's previous user is done.
            bsync();
            c.wn += Tp;
        }
        if (normed && has) {
            wait_count(fb, c.ready_op + 1, q + 1, 10);                 // 1/rms of this projection's input rows
            __threadfence_block();
        }
        if (has) epi(t0 + p0 + c.warp, acc);
    }
}

}  // namespace fwd
