// Weight and activation streams of the forward kernel: the producer threads, the
// thread that issues the tensor-core instructions, and the projection loop of the
// phase warps.
//
// Order of everything, identical on all sides: projections q = 0, 1, ... of the
// forward (four per layer, then the LM head); inside a projection the passes of
// this block (at most MAX_TILES tiles each, evenly sized); inside a pass the k
// blocks of KB columns.  Weight stage number n of the block (one k block of the
// pass's rows) uses barrier pair n % NB and the next free bytes of the ring;
// activation stage number m (XK columns) lives in stage m % XS.
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

// Placement of the stages in the byte ring: each takes the next `bytes` (a multiple of 1 KB), starting over at
// the ring's base when it would run past the end.  The producer and the MMA thread replay the same sequence.
__device__ __forceinline__ int ring_place(int &head, int bytes, int ring_bytes) {
    if (head + bytes > ring_bytes) head = 0;
    const int at = head;
    head += bytes;
    return at;
}

// Lane 0 of the W_PRODUCERS weight warps: every weight stage of the block, for the whole forward, in order;
// producer `me` issues the stages n with n % W_PRODUCERS == me (one thread alone issues a bulk copy only every
// 0.4 us or so) and replays the placement of the others.  A stage may be written once every earlier stage that
// overlaps its bytes has been released; stages are released in order, and stage n - NB before stage n is issued.
__device__ __forceinline__ void weight_producer(Ctx &c, const FwdBufs &fb, const Plan &P, int me) {
    int n = 0, tail = 0, head = 0;
    int q_s[NB], q_e[NB];
    for (int q = 0; q < n_ops(P); ++q) {
        const GemmOp &op = P.op[op_index(P, q)];
        const bf16 *wl = op.W + (size_t)op_layer(P, q) * op.lstride;
        int t0, T, k_lo, k_hi;
        op_range(op, c.cta, c.ncta, t0, T, k_lo, k_hi);
        for (int p = 0; p < n_passes(T, P.max_tiles); ++p) {
            int p0, Tp;
            pass_range(T, p, P.max_tiles, p0, Tp);
            const int bytes = Tp * 2048;                 // two 8-row atoms per tile
            for (int k = k_lo; k < k_hi; k += KB, ++n) {
                const int at = ring_place(head, bytes, c.ring_bytes), end = at + bytes;
                if (n % W_PRODUCERS == me) {
                    if (tail < n - NB) tail = n - NB;       // older stages were released before stage n - NB
                    int need = n - tail >= NB ? tail + 1 : tail;
                    for (int j = tail; j < n; ++j)
                        if (q_s[j % NB] < end && at < q_e[j % NB]) need = j + 1;
                    for (; tail < need; ++tail)
                        if (!wait_bar(fb, c.wempty + tail % NB, ((uint32_t)(tail / NB)) & 1u, 5, tail)) return;   // stop feeding
                    mbar_expect_tx(c.wfull + n % NB, (uint32_t)bytes);
                    bulk_g2s(c.ring + at, wl + ((size_t)(k >> 6) * (2 * op.MT) + 2 * (t0 + p0)) * 512, (uint32_t)bytes,
                             c.wfull + n % NB, c.policy);
                }
                q_s[n % NB] = at; q_e[n % NB] = end;
            }
        }
    }
}

// Lane 0 of warp MMA_ISSUER: the tensor-core instructions of every stage.  Per k block four MMAs of K = 16 per row
// group; the A operand is the group's part of the activation stage (128 rows are read from its base: values,
// remainders, then whatever follows in shared memory, which only reaches accumulator lanes nobody reads), the B
// operand the weight stage.  BIG: forwards with more than 32 rows (up to three row groups, each with its own
// accumulator; the stage geometry comes from the plan).
template <int NT, bool TWO, bool BIG>
__device__ __forceinline__ void mma_issuer(Ctx &c, const FwdBufs &fb, const Plan &P, int G_) {
    const int G = BIG ? G_ : 1;
    const int XS = BIG ? P.xs : x_stages(NT), XKBN = BIG ? P.xkb : XK / KB;          // stages; k blocks per stage
    const int XKB_BYTES = BIG ? P.xkb_bytes : 2 * NT * 1024, XSTAGE_BYTES = XKBN * XKB_BYTES;
    const int GROUP_BYTES = 2 * NT * 1024;
    int n = 0, head = 0, m = 0, np = 0;
    for (int q = 0; q < n_ops(P); ++q) {
        const GemmOp &op = P.op[op_index(P, q)];
        int t0, T, k_lo, k_hi;
        op_range(op, c.cta, c.ncta, t0, T, k_lo, k_hi);
        for (int p = 0; p < n_passes(T, P.max_tiles); ++p, ++np) {
            int p0, Tp;
            pass_range(T, p, P.max_tiles, p0, Tp);
            const int bytes = Tp * 2048;
            const int T0 = TWO ? min(Tp, MMA_TILES) : Tp, T1 = Tp - T0;      // tiles of the first / second accumulator
            const uint32_t idesc = umma_idesc(T0 * 16), idesc1 = umma_idesc(T1 ? T1 * 16 : 16);
            // the phase warps have copied the previous pass's accumulator out
            if (!wait_bar(fb, c.acc_empty, (((uint32_t)np) & 1u) ^ 1u, 11, np)) return;
            for (int k = k_lo; k < k_hi; k += KB, ++n) {
                const int kx = ((k - k_lo) / KB) % XKBN, xslot = m % XS;
                if (kx == 0 && !wait_bar(fb, c.xfull + xslot, ((uint32_t)(m / XS)) & 1u, 8, m)) return;
                const int at = ring_place(head, bytes, c.ring_bytes);
                if (!wait_bar(fb, c.wfull + n % NB, ((uint32_t)(n / NB)) & 1u, 9, n)) return;
                tc_fence_after();
                const uint32_t a0 = smem_u32(c.scratch + xslot * XSTAGE_BYTES + kx * XKB_BYTES), b0 = smem_u32(c.ring + at);
                const uint32_t acc = (k > k_lo) ? 1u : 0u;
                for (int g = 0; g < G; ++g) {
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16)
                        umma(c.tmem + g * P.acc_stride, umma_desc(a0 + g * GROUP_BYTES + k16 * 32), umma_desc(b0 + k16 * 32), idesc,
                             (acc || k16 > 0) ? 1u : 0u);
                }
                if (TWO && T1) {                         // (only in the kernel variant with two accumulators: the common
                                                         // variant's loop is the kernel's critical path and stays minimal)
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16)
                        umma(c.tmem + ACC_COLS, umma_desc(a0 + k16 * 32), umma_desc(b0 + T0 * 2048 + k16 * 32), idesc1,
                             (acc || k16 > 0) ? 1u : 0u);
                }
                umma_commit(c.wempty + n % NB);
                if (kx == XKBN - 1 || k + KB >= k_hi) { umma_commit(c.xempty + xslot); ++m; }
            }
            umma_commit(c.acc_full);
        }
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// inv_rms[r] = 1 / sqrt(mean(x_r^2) + eps) from the per-tile sums ssq[tile][row], in a fixed
// order (one warp, lane = row; four running sums keep the loads independent).
__device__ __forceinline__ void compute_inv(Ctx &c, const FwdBufs &fb, int dm, float eps, int row0 = 0) {
    const int ntiles = dm >> 4;
    const bool in = row0 + c.lane < MAX_ROWS;            // (the last 32-row round of a wide forward is partial)
    const float *p = fb.ssq + (in ? row0 + c.lane : 0);
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    int t = 0;
    for (; t + 4 <= ntiles; t += 4) {
        s0 += __ldcg(p + (t + 0) * MAX_ROWS);
        s1 += __ldcg(p + (t + 1) * MAX_ROWS);
        s2 += __ldcg(p + (t + 2) * MAX_ROWS);
        s3 += __ldcg(p + (t + 3) * MAX_ROWS);
    }
    for (; t < ntiles; ++t) s0 += __ldcg(p + t * MAX_ROWS);
    if (in) c.inv_rms[row0 + c.lane] = rsqrtf(((s0 + s1) + (s2 + s3)) / (float)dm + eps);
    __syncwarp();
}

// Warps X_PRODUCER .. X_PRODUCER + XS - 1: the activation stage of every XK columns, once the projection's
// inputs are complete (the phase warps raise ready_op[0] after the grid barrier): one bulk copy of a buffer that
// already has operand order.  Stage s is fed by producer s, so its generations stay in order.  A later pass of
// the same projection starts once the epilogue of the pass before is over (it uses the ring's bytes).
template <int NT, bool BIG>
__device__ __forceinline__ void activation_producer(Ctx &c, const FwdBufs &fb, const Plan &P, int me, uint64_t keep_policy) {
    const int XS = BIG ? P.xs : x_stages(NT), XKBN = BIG ? P.xkb : XK / KB;
    const int XKB_BYTES = BIG ? P.xkb_bytes : 2 * NT * 1024, XSTAGE_BYTES = XKBN * XKB_BYTES;
    if (me >= XS) return;
    int m = 0, np = 0;
    for (int q = 0; q < n_ops(P); ++q) {
        const GemmOp &op = P.op[op_index(P, q)];
        int t0, T, k_lo, k_hi;
        op_range(op, c.cta, c.ncta, t0, T, k_lo, k_hi);
        if (T == 0) continue;
        wait_count(fb, c.ready_op, q + 1, 6);
        __threadfence_block();
        asm volatile("fence.proxy.async;" ::: "memory");
        for (int p = 0; p < n_passes(T, P.max_tiles); ++p, ++np) {
            if (p > 0) {
                wait_count(fb, c.pass_done, np, 12);
                __threadfence_block();
                asm volatile("fence.proxy.async;" ::: "memory");
            }
            for (int k = k_lo; k < k_hi; k += XKBN * KB, ++m) {
                if (m % XS != me) continue;
                const int slot = m % XS, nkb = min(XKBN * KB, k_hi - k) / KB;
                if (!wait_bar(fb, c.xempty + slot, (((uint32_t)(m / XS)) & 1u) ^ 1u, 7, m)) return;
                if (c.lane == 0) {
                    const uint32_t bytes = (uint32_t)nkb * (uint32_t)XKB_BYTES;
                    mbar_expect_tx(c.xfull + slot, bytes);
                    bulk_g2s(c.scratch + slot * XSTAGE_BYTES, op.X + (size_t)(k >> 6) * (XKB_BYTES / 2), bytes, c.xfull + slot, keep_policy);
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

// One projection, run by the eight phase warps after the grid barrier that completed its inputs: per pass they
// wait for the accumulator(s), copy them piece by piece from tensor memory to shared memory (a piece: the lanes
// of one row group, values part and remainders part, and at most CH tiles of columns), and run
// epi(tile, row base, acc) for the piece's 16-row tiles, warp w taking tiles w, w + 8.
// Accumulator element (nt, i) as the epilogues see it: token row (row base) + nt*8 + 2t + (i & 1), tile column
// g + 8*(i >> 1), with g = lane / 4, t = lane % 4.  resid: rows added to the sums (the residual stream), or NULL.
template <int NT, bool TWO, bool BIG, class Epi>
__device__ __forceinline__ void gemm_op(Ctx &c, const FwdBufs &fb, const Plan &P, int q, int G_, int dm, float eps,
                                        const float *resid, int resid_ld, Epi epi) {
    const GemmOp &op = P.op[op_index(P, q)];
    const int G = BIG ? G_ : 1;
    if (threadIdx.x == 0) {
        __threadfence_block();
        c.ready_op[0] = q + 1;                 // the activation producer may start on this projection
    }
    const int opi = op_index(P, q);
    const bool normed = opi == OP_QKV || opi == OP_GU || opi == OP_HEAD;
    int t0, T, k_lo, k_hi;
    op_range(op, c.cta, c.ncta, t0, T, k_lo, k_hi);
    if (BIG && normed && T > 0) {
        // 1/rms of the input rows, by the phase warps themselves while the tensor cores work on the first pass
        // (32 rows per warp and round; in the small forwards the helper warp does this)
        for (int row0 = 32 * c.warp; row0 < G * 8 * NT; row0 += 32 * MMA_WARPS) compute_inv(c, fb, dm, eps, row0);
        bsync();
    }
    float *stage = reinterpret_cast<float *>(c.scratch);
    const int g = c.lane >> 2, t = c.lane & 3;
    constexpr int CH = NT <= 4 ? MMA_TILES : 8;             // tiles of one piece: the copy must fit the scratch
    static_assert((16 * NT + 31) / 32 * 32 * (CH * 16 + 1) * 4 <= SCRATCH_BYTES, "accumulator copy does not fit the scratch");
    for (int p = 0; p < n_passes(T, P.max_tiles); ++p) {
        int p0, Tp;
        pass_range(T, p, P.max_tiles, p0, Tp);
        wait_bar(fb, c.acc_full, ((uint32_t)c.np) & 1u, 10, c.np);
        tc_fence_after();
        const int n_acc = BIG ? G : ((TWO && Tp > MMA_TILES) ? 2 : 1);      // accumulators of this pass
        bool first = true;
        for (int ai = 0; ai < n_acc; ++ai) {
            const int a_t0 = (!BIG && ai) ? MMA_TILES : 0;                 // first tile of the pass in this accumulator
            const int a_T = BIG ? Tp : (TWO ? min(MMA_TILES, Tp - a_t0) : Tp);
            const uint32_t a_col = BIG ? (uint32_t)(ai * P.acc_stride) : (ai ? ACC_COLS : 0);
            const int rb = BIG ? ai * 8 * NT : 0;
            for (int c0 = 0; c0 < a_T; c0 += CH) {
                const int Th = min(CH, a_T - c0);
                const int C = Th * 16, pitch = C + 1;       // odd pitch: a warp's 32 lanes (rows) hit 32 banks
                const bool last = ai == n_acc - 1 && c0 + CH >= a_T;
                if (!first) bsync();                         // the copy before this one has been read
                first = false;
                {
                    const int quad = c.warp & 3;             // the accumulator lanes this warp can read: 32 quad ..
                    if (quad * 32 < 16 * NT) {
                        for (int cg = c.warp >> 2; cg * 32 < C; cg += 2) {
                            uint32_t v[32];
                            tmem_ld32(c.tmem + a_col + ((uint32_t)(quad * 32) << 16) + (uint32_t)(c0 * 16 + cg * 32), v);
                            float *row = stage + (size_t)(quad * 32 + c.lane) * pitch + cg * 32;
#pragma unroll
                            for (int jj = 0; jj < 32; ++jj)
                                if (cg * 32 + jj < C) row[jj] = __uint_as_float(v[jj]);
                        }
                    }
                }
                tc_fence_before();
                bsync();
                if (threadIdx.x == 0 && last) mbar_arrive(c.acc_empty);   // the next pass may overwrite the accumulators
                if (normed && !BIG && ai == 0 && c0 == 0) {
                    wait_count(fb, c.ready_op + 1, q + 1, 10);             // 1/rms of this projection's input rows
                    __threadfence_block();
                }
                for (int ti = c.warp; ti < Th; ti += MMA_WARPS) {
                    const int tile = t0 + p0 + a_t0 + c0 + ti;
                    float acc[NT][4];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int r = nt * 8 + 2 * t + (i & 1), cc = ti * 16 + g + 8 * (i >> 1);
                            float v = stage[(size_t)r * pitch + cc] + stage[(size_t)(8 * NT + r) * pitch + cc];
                            if (resid) {
                                const int n0 = tile * 16 + g + 8 * (i >> 1);
                                if (n0 < op.N) v += __ldcg(resid + (size_t)(rb + r) * resid_ld + n0);
                            }
                            acc[nt][i] = v;
                        }
                    epi(tile, rb, acc);
                }
            }
        }
        fence_proxy_async();                   // the copy in shared memory is read; bulk copies may overwrite it
        bsync();
        ++c.np;
        if (threadIdx.x == 0) { __threadfence_block(); *c.pass_done = c.np; }
    }
}

}  // namespace fwd
