// The forward kernel itself, the tails that take the loop's decisions (Eq. 6 /
// Eq. 7 / Algorithm 1) on the device, the host-side plan and the cooperative launch.
#pragma once
#include <algorithm>
#include <vector>

#include "fwd_attention.cuh"
#include "sampling.cuh"

namespace fwd {

// ------------------------------------------------------------------ tails (one block per sequence)

__device__ __forceinline__ float hidden_at(const Args &a, const Ctx &c, int r, int i) {
    return __ldcg(a.d.xres + (size_t)r * a.m.cfg.d_model + i) * c.inv_rms[r] * __bfloat162float(a.m.normf[i]);
}

// 1/rms of the final residual rows of sequence s, for the final RMSNorm the tails apply (MMA warps of one block).
__device__ __forceinline__ void tail_inv_rms(Ctx &c, const Args &a, int s) {
    const int dm = a.m.cfg.d_model;
    float *red = reinterpret_cast<float *>(c.scratch);
    for (int j = 0; j < c.n_rows[s]; ++j) {
        const int r = s * a.g.rps + j;
        float ss = 0.f;
        for (int i = threadIdx.x; i < dm; i += MMA_THREADS) { const float v = __ldcg(a.d.xres + (size_t)r * dm + i); ss += v * v; }
        ss = mma_block_sum(ss, red);
        if (threadIdx.x == 0) c.inv_rms[r] = rsqrtf(ss / (float)dm + a.m.cfg.rms_eps);
    }
    bsync();
}

// End of one draft forward (Eq. 6): y_i, h_i queued for the pre-verification model, cache length.
__device__ __forceinline__ void tail_draft(Ctx &c, const Args &a, int s) {
    const DevPtrs &d = a.d;
    SeqState &st = d.st[s];
    const int n_in = c.n_rows[s], dm = a.m.cfg.d_model;
    if (n_in == 0) return;
    const int gamma = st.gamma, n_pend = st.n_pend, r_last = s * a.g.rps + n_in - 1;
    int y_new = 0;
    if (st.mode == PACER_SAMPLE)                          // y_i ~ q_i by the Gumbel-max rule at the token's position
        y_new = gumbel_argmax(d.draft_logits + ((size_t)s * d.gamma_cap + gamma) * a.m.cfg.vocab, a.m.cfg.vocab, st.seed,
                              st.P + gamma, s, TAG_DRAFT, MMA_THREADS, reinterpret_cast<BestD *>(c.scratch), true);
    const bool queue = !st.sched;                        // with prescribed windows nothing is pre-verified
    for (int jj = 0; queue && jj < n_in; ++jj) {
        float *dst = d.hpend + ((size_t)s * (d.block_b + 1) + n_pend + jj) * dm;
        for (int i = threadIdx.x; i < dm; i += MMA_THREADS) dst[i] = hidden_at(a, c, s * a.g.rps + jj, i);
    }
    bsync();
    if (threadIdx.x == 0) {
        for (int jj = 0; queue && jj < n_in; ++jj)
            d.hpend_e[s * (d.block_b + 1) + n_pend + jj] = (jj == n_in - 1) ? gamma + 1 : 0;
        d.y[(size_t)s * d.gamma_cap + gamma] = st.mode == PACER_SAMPLE ? y_new : d.row_arg[r_last];
        if (queue) st.n_pend = n_pend + n_in;
        st.gamma = gamma + 1;
        st.len_D += n_in;
        st.n_draft_fwd += 1;
    }
}

// End of a pre-verification call (Eq. 7 + the block test of Algorithm 1).
__device__ __forceinline__ void tail_mb(Ctx &c, const Args &a, int s) {
    const DevPtrs &d = a.d;
    SeqState &st = d.st[s];
    const int n = c.n_rows[s], dm = a.m.cfg.d_model;
    if (n == 0) return;
    float *red = reinterpret_cast<float *>(c.scratch);
    for (int j = 0; j < n; ++j) {
        const int r = s * a.g.rps + j, e = c.row_tok[r];
        if (e == 0) continue;
        float z0 = 0.f, z1 = 0.f;
        for (int i = threadIdx.x; i < dm; i += MMA_THREADS) {
            const float hv = hidden_at(a, c, r, i);
            z0 += hv * __bfloat162float(a.m.head_b[i]);
            z1 += hv * __bfloat162float(a.m.head_b[dm + i]);
        }
        z0 = mma_block_sum(z0, red);
        z1 = mma_block_sum(z1, red);
        if (threadIdx.x == 0) d.alpha[(size_t)s * d.gamma_cap + e - 1] = 1.f / (1.f + expf(z0 - z1));
    }
    bsync();
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
        if (gamma == b) {                     // first call of the step: where its drafts begin in the cache
            int n_hist = 0;
            while (n_hist < n && c.row_tok[s * a.g.rps + n_hist] == 0) ++n_hist;
            st.mb_start = st.len_B + n_hist;
        }
        st.len_B += n;
        st.n_pend = 0;
        st.n_mb_calls += 1;
    }
}

// End of a prefill chunk: the caches grew; the draft's hidden rows are the
// history rows the pre-verification model is prefilled with.
__device__ __forceinline__ void tail_prefill(Ctx &c, const Args &a, int s, int which) {
    const DevPtrs &d = a.d;
    const int n = c.n_rows[s], dm = a.m.cfg.d_model;
    if (n == 0) return;
    if (which == PACER_DRAFT)
        for (int j = 0; j < n; ++j) {
            const int r = s * a.g.rps + j;
            for (int i = threadIdx.x; i < dm; i += MMA_THREADS) d.hidden[(size_t)r * dm + i] = hidden_at(a, c, r, i);
        }
    if (threadIdx.x == 0) {
        SeqState &st = d.st[s];
        if (which == PACER_TARGET) st.len_T += n;
        else if (which == PACER_DRAFT) st.len_D += n;
        else st.len_B += n;
    }
}

// End of one autoregressive target step (Eq. 1).
__device__ __forceinline__ void tail_ar(Ctx &c, const Args &a, int s) {
    if (c.n_rows[s] == 0) return;
    const DevPtrs &d = a.d;
    SeqState &st = d.st[s];
    int tok = d.row_arg[s * a.g.rps];
    if (st.mode == PACER_SAMPLE)
        tok = gumbel_argmax(d.verify_logits + (size_t)s * (d.gamma_cap + 1) * a.m.cfg.vocab, a.m.cfg.vocab, st.seed, st.P, s,
                            TAG_NEXT, MMA_THREADS, reinterpret_cast<BestD *>(c.scratch), true);
    if (threadIdx.x != 0) return;
    d.x[(size_t)s * d.max_ctx + st.P] = tok;
    st.P += 1;
    st.len_T += 1;
    st.n_target_fwd += 1;
    st.n_steps += 1;
    if (st.P - st.n_prompt >= st.max_new) st.finished = 1;
}

// ------------------------------------------------------------------ the kernel

template <int NT, bool TWO, bool BIG>
__global__ void __launch_bounds__(THREADS, 1) k_forward(const __grid_constant__ Args a, const int which) {
    extern __shared__ __align__(1024) unsigned char smem[];
    if (smem_u32(smem) & 1023u) {           // the swizzled operand layout needs this alignment (the same in every block)
        if (threadIdx.x == 0) atomicCAS(a.fb.abort_flag, 0, 13);
        return;
    }
    Ctx c;
    c.warp = threadIdx.x >> 5; c.lane = threadIdx.x & 31; c.cta = blockIdx.x; c.ncta = gridDim.x;
    c.scratch = smem;
    c.ring = smem + a.P.scratch_bytes;
    c.ring_bytes = a.P.ring_bytes;
    unsigned char *misc = smem + a.P.scratch_bytes + a.P.ring_bytes;
    c.wfull = reinterpret_cast<uint64_t *>(misc);                            // NB
    c.wempty = c.wfull + NB;                                                 // NB
    c.xfull = c.wempty + NB;                                                 // XS_MAX
    c.xempty = c.xfull + XS_MAX;                                             // XS_MAX
    c.acc_full = c.xempty + XS_MAX;
    c.acc_empty = c.acc_full + 1;                                            // ends at 8 * (2*NB + 2*XS_MAX + 2) = 320
    static_assert(8 * (2 * NB + 2 * XS_MAX + 2) <= 320, "barriers overlap the row tables");
    c.row_pos = reinterpret_cast<int32_t *>(misc + 320);                     // four tables of MAX_ROWS words
    c.row_tok = c.row_pos + MAX_ROWS;
    c.inv_rms = reinterpret_cast<float *>(c.row_tok + MAX_ROWS);
    int32_t *bias_at = reinterpret_cast<int32_t *>(c.inv_rms + MAX_ROWS);
    float **row_dst = reinterpret_cast<float **>(misc + 320 + 16 * MAX_ROWS); // [MAX_ROWS] pointers
    unsigned char *tail_misc = misc + 320 + 24 * MAX_ROWS;
    c.n_rows = reinterpret_cast<int32_t *>(tail_misc);                       // [MAX_SEQ]
    c.key_start = c.n_rows + MAX_SEQ;                                        // [MAX_SEQ]
    c.ready_op = reinterpret_cast<volatile int32_t *>(c.key_start + MAX_SEQ); // 2 words
    c.flag = reinterpret_cast<int32_t *>(tail_misc + 8 * MAX_SEQ + 16);      // 4 words
    Top2 *top_sm = reinterpret_cast<Top2 *>(tail_misc + 8 * MAX_SEQ + 32);   // [8]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tail_misc + 8 * MAX_SEQ + 160);
    c.pass_done = reinterpret_cast<volatile int32_t *>(tail_misc + 8 * MAX_SEQ + 164);
    static_assert(320 + 24 * MAX_ROWS + 8 * MAX_SEQ + 168 <= MISC_BYTES, "row tables do not fit");
    c.bar_target = 0;
    c.np = 0;
    c.tmem = 0;
    c.policy = policy_evict_first();
    const DevPtrs &d = a.d;
    const ModelDev &m = a.m;
    const Geom &g = a.g;
    const int kind = a.kind;
    constexpr int TMEM_COLS = (TWO || BIG) ? 2 * ACC_COLS : ACC_COLS;

    // rows of this forward, from the sequence state
    if (threadIdx.x < MAX_ROWS) {
        const int r = threadIdx.x;
        int pos = -1, tok = 0;
        if (r < g.rtot) {
            const RowDesc rd = row_desc(kind, d, r / g.rps, r % g.rps, a.aux);
            if (rd.active) { pos = rd.pos; tok = rd.tok; }
        }
        c.row_pos[r] = pos; c.row_tok[r] = tok;
    }
    __syncthreads();
    if (threadIdx.x < MAX_SEQ) {
        const int s = threadIdx.x;
        int n = 0, ks = 0;
        if (s < g.batch) {
            for (int j = 0; j < g.rps; ++j) n += c.row_pos[s * g.rps + j] >= 0;
            if (kind == KIND_MB && d.mb_scope != 0 && n > 0) {
                // restricted attention context: from the first draft row of the block, or of the step
                int n_hist = 0;
                while (n_hist < n && c.row_tok[s * g.rps + n_hist] == 0) ++n_hist;
                const int first = c.row_pos[s * g.rps] + n_hist;
                ks = (d.mb_scope == 2 || d.st[s].gamma == d.block_b) ? first : d.st[s].mb_start;
            }
        }
        c.n_rows[s] = n;
        c.key_start[s] = ks;
    }
    __syncthreads();
    int any = 0;
    for (int s = 0; s < g.batch; ++s) any |= c.n_rows[s];
    if (c.cta == 0 && threadIdx.x < MAX_ROWS) {
        if (threadIdx.x < g.batch && threadIdx.x < MAX_SEQ) d.n_rows[threadIdx.x] = c.n_rows[threadIdx.x];
        if (threadIdx.x < g.rtot) { d.row_pos[threadIdx.x] = c.row_pos[threadIdx.x]; d.row_tok[threadIdx.x] = c.row_tok[threadIdx.x]; }
    }
    if (!any) return;                       // every sequence idles: the same decision in every block

    if (threadIdx.x < MAX_ROWS) {           // where the LM-head rows go
        const int r = threadIdx.x;
        float *dst = nullptr;
        int b = -1;
        if (r < g.rtot && c.row_pos[r] >= 0 && a.P.has_head) {
            const int s = r / g.rps, j = r - s * g.rps, V = m.cfg.vocab;
            if (kind == KIND_DRAFT) {
                if (j == c.n_rows[s] - 1) dst = d.draft_logits + ((size_t)s * d.gamma_cap + d.st[s].gamma) * V;
            } else {
                dst = d.verify_logits + ((size_t)s * (d.gamma_cap + 1) + j) * V;
            }
            if (m.succ) b = m.succ[c.row_tok[r]];
        }
        row_dst[r] = dst; bias_at[r] = b;
    }
    if (threadIdx.x == 0) {
        const unsigned long long v = ld_acquire_u64(a.fb.bar);
        c.bar_target = v / (unsigned long long)c.ncta * (unsigned long long)c.ncta;
        for (int i = 0; i < NB; ++i) { mbar_init(c.wfull + i, 1); mbar_init(c.wempty + i, 1); }
        for (int i = 0; i < XS_MAX; ++i) { mbar_init(c.xfull + i, 1); mbar_init(c.xempty + i, 1); }
        mbar_init(c.acc_full, 1); mbar_init(c.acc_empty, 1);
        c.ready_op[0] = 0; c.ready_op[1] = 0;
        *c.pass_done = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (c.warp == MMA_ISSUER) {             // the accumulator's tensor memory, held until the end of the kernel
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    c.tmem = *tmem_slot;

    // the producer warps live in their streams until the forward's last stage
    if (c.warp == W_PRODUCER || c.warp == 10 || c.warp == 11) {
        if (c.lane == 0) weight_producer(c, a.fb, a.P, c.warp == W_PRODUCER ? 0 : c.warp - 9);
        return;
    }
    if (c.warp == MMA_ISSUER) {
        if (c.lane == 0) mma_issuer<NT, TWO, BIG>(c, a.fb, a.P, g.G);
        __syncwarp();
        asm volatile("bar.sync 2, 288;" ::: "memory");        // the phase warps have read their last accumulator
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(c.tmem), "r"(TMEM_COLS) : "memory");
        return;
    }
    if (c.warp == X_PRODUCER + X_PRODUCERS - 1) {           // (in the wide forwards the phase warps compute 1/rms themselves)
        if (!BIG) helper_warp(c, a.fb, a.P, m.cfg.d_model, m.cfg.rms_eps);
        return;
    }
    if (c.warp >= X_PRODUCER) {
        uint64_t keep;
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep));
        activation_producer<NT, BIG>(c, a.fb, a.P, c.warp - X_PRODUCER, keep);
        return;
    }

    const int dm = m.cfg.d_model;
    int n_stamp = 0;
    auto stamp = [&]() {
        if (a.fb.prof && threadIdx.x == 0 && n_stamp < PROF_STAMPS)
            a.fb.prof[(size_t)c.cta * PROF_STAMPS + n_stamp++] = globaltimer_ns();
    };
    stamp();
    phase_begin(c, a);
    stamp();
    grid_barrier(c, a.fb);
    stamp();

    const int L = a.P.n_layers;
    for (int l = 0; l < L; ++l) {
        {
            const int slice = op_slice(a.P.op[OP_QKV], c.cta, c.ncta);
            gemm_op<NT, TWO, BIG>(c, a.fb, a.P, 4 * l + OP_QKV, g.G, dm, m.cfg.rms_eps, nullptr, 0,
                        [&](int tile, int rb, float (&acc)[NT][4]) { epi_qkv<NT>(c, a, slice, tile, rb, acc); });
        }
        stamp();
        grid_barrier(c, a.fb);
        stamp();
        const int nsplit = attention_splits(c, a);
        phase_attention(c, a, l, nsplit);
        stamp();
        grid_barrier(c, a.fb);
        if (nsplit > 1) {                       // the same decision in every block
            phase_attention_merge(c, a, nsplit);
            grid_barrier(c, a.fb);
        }
        stamp();
        {
            const GemmOp &op = a.P.op[OP_O];
            const bf16 *gain_next = m.norm2 + (size_t)l * dm;
            if (op.S == 1) {
                gemm_op<NT, TWO, BIG>(c, a.fb, a.P, 4 * l + OP_O, g.G, dm, m.cfg.rms_eps, d.xres, dm,
                            [&](int tile, int rb, float (&acc)[NT][4]) { epi_residual<NT>(c, a, gain_next, tile, rb, acc); });
            } else {
                const int slice = op_slice(op, c.cta, c.ncta);
                gemm_op<NT, TWO, BIG>(c, a.fb, a.P, 4 * l + OP_O, g.G, dm, m.cfg.rms_eps, nullptr, 0,
                            [&](int tile, int rb, float (&acc)[NT][4]) { epi_partial<NT>(c, a, op, slice, tile, rb, acc); });
            }
            stamp();
            grid_barrier(c, a.fb);
            if (op.S > 1) {
                phase_residual<NT, BIG>(c, a, op, gain_next);
                grid_barrier(c, a.fb);
            }
            stamp();
        }
        gemm_op<NT, TWO, BIG>(c, a.fb, a.P, 4 * l + OP_GU, g.G, dm, m.cfg.rms_eps, nullptr, 0, [&](int tile, int rb, float (&acc)[NT][4]) { epi_swiglu<NT>(c, a, tile, rb, acc); });
        stamp();
        grid_barrier(c, a.fb);
        stamp();
        {
            const GemmOp &op = a.P.op[OP_DOWN];
            const bf16 *gain_next = l + 1 < L ? m.norm1 + (size_t)(l + 1) * dm : m.normf;
            if (op.S == 1) {
                gemm_op<NT, TWO, BIG>(c, a.fb, a.P, 4 * l + OP_DOWN, g.G, dm, m.cfg.rms_eps, d.xres, dm,
                            [&](int tile, int rb, float (&acc)[NT][4]) { epi_residual<NT>(c, a, gain_next, tile, rb, acc); });
            } else {
                const int slice = op_slice(op, c.cta, c.ncta);
                gemm_op<NT, TWO, BIG>(c, a.fb, a.P, 4 * l + OP_DOWN, g.G, dm, m.cfg.rms_eps, nullptr, 0,
                            [&](int tile, int rb, float (&acc)[NT][4]) { epi_partial<NT>(c, a, op, slice, tile, rb, acc); });
            }
            stamp();
            grid_barrier(c, a.fb);
            if (op.S > 1) {
                phase_residual<NT, BIG>(c, a, op, gain_next);
                grid_barrier(c, a.fb);
            }
            stamp();
        }
    }
    if (a.P.has_head) {
        gemm_op<NT, TWO, BIG>(c, a.fb, a.P, 4 * L, g.G, dm, m.cfg.rms_eps, nullptr, 0,
                    [&](int tile, int rb, float (&acc)[NT][4]) { epi_head<NT>(c, a, row_dst, bias_at, tile, rb, acc); });
        stamp();
        grid_barrier(c, a.fb);
        stamp();
        if (kind == KIND_VERIFY) {
            if (c.cta < g.rtot && row_dst[c.cta]) head_row_argmax(a, c.cta, top_sm);
            if (a.aux) {                    // whole-loop runs, greedy: acceptance (Eq. 5), commit and rollback right here
                grid_barrier(c, a.fb);
                if (c.cta < g.batch && threadIdx.x == 0) accept_greedy_seq(d, g, c.cta);
            }
        } else if (c.cta < g.batch && c.n_rows[c.cta] > 0) {
            head_row_argmax(a, c.cta * g.rps + c.n_rows[c.cta] - 1, top_sm);
        }
    }
    if (c.cta < g.batch && kind != KIND_VERIFY) {
        if (kind != KIND_AR) tail_inv_rms(c, a, c.cta);     // the tails below apply the final RMSNorm themselves
        if (kind == KIND_DRAFT) tail_draft(c, a, c.cta);
        else if (kind == KIND_MB) tail_mb(c, a, c.cta);
        else if (kind == KIND_AR) tail_ar(c, a, c.cta);
        else if (kind == KIND_PREFILL || kind == KIND_PREFILL_B) tail_prefill(c, a, c.cta, which);
    }
    stamp();
    tc_fence_before();
    asm volatile("bar.sync 2, 288;" ::: "memory");            // lets the owner release the tensor memory
}

}  // namespace fwd

// ------------------------------------------------------------------ host: plan and launch

namespace fwd {

static inline Plan make_plan(const ModelDev &m, const DevPtrs &d, const FwdBufs &fb, int ncta, bool has_head, const Geom &geom) {
    Plan P;
    memset(&P, 0, sizeof P);
    const pacer_model_cfg &k = m.cfg;
    const long long dm = k.d_model, F = k.d_ffn, hh = (long long)k.n_heads * m.hd;
    int rot = 0;
    auto set = [&](int i, const bf16 *w, const bf16 *x, int N, int K, int MT) {
        GemmOp &o = P.op[i];
        o.W = w; o.X = x; o.N = N; o.K = K; o.MT = MT;
        o.lstride = (long long)(K / KB) * (2 * MT) * 512;
        o.S = 1;
        // few tiles and enough bytes to be bandwidth bound: also cut along k, so that a block needs less of the
        // activations (a small projection is latency bound and better off without the extra pass and barrier)
        // (the wider a block's row range, the larger its stages: a stage costs the issuing threads about 0.4 us
        // whatever its size).  As many slices as keep a block's share within one pass, four at most.
        if ((i == OP_QKV || i == OP_O || i == OP_DOWN) && (long long)N * K * 2 >= (16ll << 20)) {
            const int nks = K / (8 * KB);                    // a slice keeps at least 512 columns
            for (int sdiv = 2; sdiv <= 4; ++sdiv)
                if (ncta % sdiv == 0 && sdiv <= nks && (MT + ncta / sdiv - 1) / (ncta / sdiv) <= MMA_TILES) o.S = sdiv;
        } else if (((i == OP_DOWN && K >= 32 * KB) || (i == OP_O && K >= 24 * KB)) && MT < ncta && ncta % 4 == 0) {
            // a small model's down (or attention-output) projection: one or two tiles per block over a long k
            // range is a chain of K / 64 stages of 0.3 - 0.4 us each, longer than the reduction pass that four
            // k slices cost
            o.S = 4;
        }
        o.rot = rot;
        rot = (rot + (MT % (ncta / o.S)) * o.S) % ncta;       // the next projection's extra tiles go to other blocks
    };
    set(OP_QKV, m.wt[OP_QKV], fb.xg, m.qrows, (int)dm, (m.qrows + 15) / 16);
    set(OP_O, m.wt[OP_O], d.att, (int)dm, (int)hh, ((int)dm + 15) / 16);
    set(OP_GU, m.wt[OP_GU], fb.xg, (int)(2 * F), (int)dm, ((int)F + 7) / 8);
    set(OP_DOWN, m.wt[OP_DOWN], d.act, (int)dm, (int)F, ((int)dm + 15) / 16);
    set(OP_HEAD, m.wt[OP_HEAD], fb.xg, k.vocab, (int)dm, (k.vocab + 15) / 16);
    P.op[OP_HEAD].lstride = 0;
    // one pass per projection where N = 256 allows it; a model in which some block has up to twice as many tiles
    // runs the kernel variant with two accumulators (the activations are then still read once)
    P.max_tiles = MMA_TILES;
    const bool big = geom.nt > 4;
    for (int i = 0; i < N_OPS && !big; ++i) {
        if (i == OP_HEAD && !has_head) continue;
        const GemmOp &o = P.op[i];
        const int groups = ncta / o.S, per_block = (o.MT + groups - 1) / groups;
        if (per_block > MMA_TILES && per_block <= MAX_TILES) P.max_tiles = MAX_TILES;
    }
    // shared memory: the forwards with at most 32 rows keep 88 KB of scratch (activation stages of 256 k columns
    // in front) and the large weight ring; the wide ones stage one k block of all row groups at a time, three
    // stages deep, and leave the rest to the weight ring
    P.xkb_bytes = 2 * geom.nt * geom.G * 1024;
    if (!big) {
        P.xkb = XK / KB; P.xs = x_stages(geom.nt);
        P.scratch_bytes = SCRATCH_BYTES; P.ring_bytes = RING_BYTES;
        P.acc_stride = 0;
    } else {
        P.xkb = std::max(1, std::min(XK / KB, (32 * 1024) / P.xkb_bytes));
        P.xs = std::max(1, std::min(XS_MAX, BIG_XBYTES / (P.xkb * P.xkb_bytes)));
        P.scratch_bytes = std::max(SCRATCH_BYTES, P.xs * P.xkb * P.xkb_bytes);
        P.ring_bytes = SCRATCH_BYTES + RING_BYTES - P.scratch_bytes;
        P.acc_stride = geom.G == 3 ? 160 : ACC_COLS;
        if (geom.G == 3) P.max_tiles = 10;
    }
    P.n_layers = k.n_layers;
    P.has_head = has_head ? 1 : 0;
    return P;
}

template <int NT, bool TWO, bool BIG>
static inline cudaError_t launch_nt(const Args &a, int which, int ncta, cudaStream_t st) {
    static bool attr_set[64] = {};           // the opt-in is per device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(k_forward<NT, TWO, BIG>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    void *params[] = {(void *)&a, (void *)&which};
    return cudaLaunchCooperativeKernel((const void *)k_forward<NT, TWO, BIG>, dim3(ncta), dim3(THREADS), params, SMEM_BYTES, st);
}

// The variant with two accumulators runs the models in which some block has more than MMA_TILES tiles of a
// projection; the wide variants (6 or 8 tiles per row group, up to three groups) the forwards with more than 32 rows.
static inline cudaError_t launch(const Args &a, int which, int ncta, cudaStream_t st) {
    const bool two = a.P.max_tiles > MMA_TILES;
    switch (a.g.nt) {
        case 1: return two ? launch_nt<1, true, false>(a, which, ncta, st) : launch_nt<1, false, false>(a, which, ncta, st);
        case 2: return two ? launch_nt<2, true, false>(a, which, ncta, st) : launch_nt<2, false, false>(a, which, ncta, st);
        case 3: return two ? launch_nt<3, true, false>(a, which, ncta, st) : launch_nt<3, false, false>(a, which, ncta, st);
        case 4: return two ? launch_nt<4, true, false>(a, which, ncta, st) : launch_nt<4, false, false>(a, which, ncta, st);
        case 6: return launch_nt<6, false, true>(a, which, ncta, st);
        case 8: return launch_nt<8, false, true>(a, which, ncta, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace fwd
