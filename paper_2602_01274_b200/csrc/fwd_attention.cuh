// Attention phase of the forward kernel: rotary embedding of the new q/k rows,
// append of k/v to the cache, and causal attention of the new rows over the
// cache, on tensor cores.  q, k, v and the probabilities enter the MMAs as split
// bf16 (value + rounding remainder, see store_split), and the cache keeps both
// parts of k and v: single bf16 operands here alone put 0.14 of error on the
// logits of a 32-layer model of width 4096.  Work items are (sequence, head,
// key-range split).  Inside an item the eight MMA warps split the keys in steps
// of 8 (and the two 16-row query tiles when there are more than 16 rows); every
// warp keeps a running (max, sum, output) per row, FlashAttention style.  The
// warps' results are merged through shared memory into the item's partial; after
// a grid barrier the splits of every (sequence, head, row) are merged by one warp
// each into the attention output, in the operand order the output projection reads.
#pragma once
#include "fwd_phases.cuh"

namespace fwd {

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void *smem_row) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(smem_row)));
}

// Geometry of the shared-memory scratch during an attention item.  "Planes": [0] the bf16 values, [1] the remainders.
template <int HD>
struct AttSmem {
    static constexpr int QP = HD * 2 + 64;   // bytes between query rows (conflict-free 16-byte reads of rows g, g+8)
    static constexpr int VP = HD * 2 + 16;   // bytes between the rows of a V step (conflict-free ldmatrix)
    static constexpr int PW = HD + 2;        // floats of a partial row: values, running max, running sum
    static constexpr int Q_OFF = 0;                           // [2 planes][32][QP] q, scaled and rotated
    static constexpr int KN_OFF = 2 * 32 * QP;                // [2 planes][32][HD] new keys as cached
    static constexpr int VN_OFF = KN_OFF + 2 * 32 * HD * 2;   // [2 planes][32][HD] new values as cached
    static constexpr int VS_OFF = VN_OFF + 2 * 32 * HD * 2;   // [8 warps][16][VP] V of the current step: 8 keys x 2 planes
    static constexpr int END = VS_OFF + MMA_WARPS * 16 * VP;
    static_assert(END <= SCRATCH_BYTES, "attention staging does not fit the scratch");
    static_assert((MMA_WARPS * 16 * PW + 32 * MMA_WARPS + 64) * 4 <= SCRATCH_BYTES, "attention merge buffer does not fit the scratch");
};

__device__ __forceinline__ void split_bf16(float v, bf16 &hi, bf16 &lo) {
    hi = __float2bfloat16(v);
    lo = __float2bfloat16(v - __bfloat162float(hi));
}

// Rotary embedding of the new rows of one item: q (scaled) of its query rows to shared memory; k, v of the kv head as
// the cache holds them, to shared memory and, by one item per kv head, to the cache.  All as split bf16.
// Query rows are VIRTUAL rows: with grouped-query attention the `group` query heads of a kv head times the n_r rows
// of the sequence are numbered v = (head within the group) * n_r + row, and an item takes 32 of them (vbase ..
// vbase + nv - 1), so that the keys of a kv head are read once for a full 32-row tile pair whatever n_r is; without
// grouping v is the row itself.  Local row lv of the item is virtual row vbase + lv; fresh key/value row lv is row
// lv of the sequence.
// KV = false (forwards with more than 32 rows per sequence): only the query rows are staged; the new keys and values
// went to the cache in a pass of their own (attention_append) and are read from there.
template <int HD, bool GQA, bool KV>
__device__ __forceinline__ void attention_rows(Ctx &c, const Args &a, int layer, int seq, int kh, int vbase, int nv, bool writer) {
    using SM = AttSmem<HD>;
    constexpr int half = HD / 2;
    const DevPtrs &d = a.d;
    const ModelDev &m = a.m;
    const int H = m.cfg.n_heads, Hkv = m.cfg.n_kv_heads, group = GQA ? H / Hkv : 1, qrows = m.qrows;
    const int n_r = c.n_rows[seq], r_base = seq * a.g.rps, pos0 = c.row_pos[r_base];
    bf16 *kn = reinterpret_cast<bf16 *>(c.scratch + SM::KN_OFF), *vn = reinterpret_cast<bf16 *>(c.scratch + SM::VN_OFF);
    const size_t cbase = (((size_t)layer * d.max_batch + seq) * Hkv + kh) * (size_t)d.max_ctx * HD;
    const float scale = rsqrtf((float)HD);
    // The projection may have been cut along k: every value is the sum of the slices' shares.  Five elements per
    // thread at a time, all their loads issued before the first use (the phase is bound by load latency).
    const int S = a.P.op[OP_QKV].S;
    const size_t sl = (size_t)MAX_ROWS * qrows;
    constexpr int U = 5;                                 // 17 rows of 128 channels are one batch
    const int n_act = (GQA ? (KV ? max(nv, n_r) : nv) : n_r) * half;
    for (int i = nv * half + threadIdx.x; i < 32 * half; i += MMA_THREADS) {     // idle query rows are zeros
        const int j = i / half, ii = i - j * half;
        bf16 *qrow = reinterpret_cast<bf16 *>(c.scratch + SM::Q_OFF + j * SM::QP);
        bf16 *qrow_lo = reinterpret_cast<bf16 *>(c.scratch + SM::Q_OFF + (32 + j) * SM::QP);
        qrow[ii] = qrow_lo[ii] = __float2bfloat16(0.f);
        qrow[ii + half] = qrow_lo[ii + half] = __float2bfloat16(0.f);
    }
    for (int i0 = threadIdx.x; i0 < n_act; i0 += U * MMA_THREADS) {
        float part[U][2][6];
        float2 csq[U], csk[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = i0 + u * MMA_THREADS, lv = i / half, ii = i - lv * half;
            const bool onk = KV && lv < n_r, onq = GQA ? lv < nv : onk;
            int h = kh, jq = lv;                                 // query row lv: head and row of the sequence
            if (GQA) { const int v = vbase + lv, hq = v / n_r; jq = v - hq * n_r; h = kh * group + hq; }
            const float *rowk = a.fb.qkv + (size_t)(r_base + (onk ? lv : 0)) * qrows;
            const float *rowq = GQA ? a.fb.qkv + (size_t)(r_base + (onq ? jq : 0)) * qrows : rowk;
            const int col[6] = {h * HD + ii, h * HD + ii + half, (H + kh) * HD + ii, (H + kh) * HD + ii + half,
                                (H + Hkv + kh) * HD + ii, (H + Hkv + kh) * HD + ii + half};
            csq[u] = onq ? m.rope[(size_t)(pos0 + jq) * half + ii] : make_float2(0.f, 0.f);
            csk[u] = !GQA ? csq[u] : (onk ? m.rope[(size_t)(pos0 + lv) * half + ii] : make_float2(0.f, 0.f));
#pragma unroll
            for (int s = 0; s < 2; ++s)
#pragma unroll
                for (int e = 0; e < 6; ++e)
                    part[u][s][e] = ((e < 2 ? onq : onk) && s < S) ? __ldcg((e < 2 ? rowq : rowk) + s * sl + col[e]) : 0.f;
            if (S > 2) {                                         // slices 2, 3: a second wave of loads
#pragma unroll
                for (int e = 0; e < 6; ++e) {
                    if (!(e < 2 ? onq : onk)) continue;
                    const float *row = e < 2 ? rowq : rowk;
                    const float p2 = __ldcg(row + 2 * sl + col[e]), p3 = S > 3 ? __ldcg(row + 3 * sl + col[e]) : 0.f;
                    part[u][0][e] += p2; part[u][1][e] += p3;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = i0 + u * MMA_THREADS, lv = i / half, ii = i - lv * half;
            if (i >= n_act) continue;
            float in[6];
#pragma unroll
            for (int e = 0; e < 6; ++e) in[e] = part[u][0][e] + part[u][1][e];
            if (GQA ? lv < nv : true) {
                bf16 *qrow = reinterpret_cast<bf16 *>(c.scratch + SM::Q_OFF + lv * SM::QP);
                bf16 *qrow_lo = reinterpret_cast<bf16 *>(c.scratch + SM::Q_OFF + (32 + lv) * SM::QP);
                const float qa = in[0], qb = in[1];
                split_bf16((qa * csq[u].x - qb * csq[u].y) * scale, qrow[ii], qrow_lo[ii]);
                split_bf16((qb * csq[u].x + qa * csq[u].y) * scale, qrow[ii + half], qrow_lo[ii + half]);
            }
            if (KV && (GQA ? lv < n_r : true)) {
                const int j = lv, pos = pos0 + j;
                const float ka = in[2], kb = in[3];
                bf16 k0, k0l, k1, k1l, v0, v0l, v1, v1l;
                split_bf16(ka * csk[u].x - kb * csk[u].y, k0, k0l);
                split_bf16(kb * csk[u].x + ka * csk[u].y, k1, k1l);
                split_bf16(in[4], v0, v0l);
                split_bf16(in[5], v1, v1l);
                kn[j * HD + ii] = k0; kn[j * HD + ii + half] = k1;
                kn[(32 + j) * HD + ii] = k0l; kn[(32 + j) * HD + ii + half] = k1l;
                vn[j * HD + ii] = v0; vn[j * HD + ii + half] = v1;
                vn[(32 + j) * HD + ii] = v0l; vn[(32 + j) * HD + ii + half] = v1l;
                if (writer) {
                    bf16 *kc = m.kcache + cbase + (size_t)pos * HD, *vc = m.vcache + cbase + (size_t)pos * HD;
                    kc[ii] = k0; kc[ii + half] = k1;
                    kc[m.kv_lo + ii] = k0l; kc[m.kv_lo + ii + half] = k1l;
                    vc[ii] = v0; vc[ii + half] = v1;
                    vc[m.kv_lo + ii] = v0l; vc[m.kv_lo + ii + half] = v1l;
                }
            }
        }
    }
}

// Forwards with more than 32 rows per sequence (prompt chunks): rotary embedding of the new k rows jbase .. jbase+31
// of (seq, kv head) and append of k, v to the cache as split bf16.  The attention items that follow a grid barrier
// read every key from the cache, the new ones under a causal mask.
template <int HD>
__device__ __forceinline__ void attention_append(Ctx &c, const Args &a, int layer, int seq, int kh, int jbase) {
    constexpr int half = HD / 2;
    const DevPtrs &d = a.d;
    const ModelDev &m = a.m;
    const int H = m.cfg.n_heads, Hkv = m.cfg.n_kv_heads, qrows = m.qrows;
    const int n_r = c.n_rows[seq], r_base = seq * a.g.rps, pos0 = c.row_pos[r_base];
    const size_t cbase = (((size_t)layer * d.max_batch + seq) * Hkv + kh) * (size_t)d.max_ctx * HD;
    const int S = a.P.op[OP_QKV].S;
    const size_t sl = (size_t)MAX_ROWS * qrows;
    const int n_el = min(32, n_r - jbase) * half;
    for (int i = threadIdx.x; i < n_el; i += MMA_THREADS) {
        const int j = jbase + i / half, ii = i % half, pos = pos0 + j;
        const float *row = a.fb.qkv + (size_t)(r_base + j) * qrows;
        const int col[4] = {(H + kh) * HD + ii, (H + kh) * HD + ii + half, (H + Hkv + kh) * HD + ii, (H + Hkv + kh) * HD + ii + half};
        float in[4] = {0.f, 0.f, 0.f, 0.f};
        for (int s_ = 0; s_ < S; ++s_)
#pragma unroll
            for (int e = 0; e < 4; ++e) in[e] += __ldcg(row + s_ * sl + col[e]);
        const float2 cs = m.rope[(size_t)pos * half + ii];
        bf16 k0, k0l, k1, k1l, v0, v0l, v1, v1l;
        split_bf16(in[0] * cs.x - in[1] * cs.y, k0, k0l);
        split_bf16(in[1] * cs.x + in[0] * cs.y, k1, k1l);
        split_bf16(in[2], v0, v0l);
        split_bf16(in[3], v1, v1l);
        bf16 *kc = m.kcache + cbase + (size_t)pos * HD, *vc = m.vcache + cbase + (size_t)pos * HD;
        kc[ii] = k0; kc[ii + half] = k1;
        kc[m.kv_lo + ii] = k0l; kc[m.kv_lo + ii + half] = k1l;
        vc[ii] = v0; vc[ii + half] = v1;
        vc[m.kv_lo + ii] = v0l; vc[m.kv_lo + ii + half] = v1l;
    }
}

// L2 prefetch of the cached K and V rows (values and remainders) of step st of this warp.  The first ATT_PF steps
// are prefetched before the new rows are prepared, every later step ATT_PF steps ahead inside the key loop: the
// loop is a chain of dependent loads, which then hit L2 instead of HBM (a burst of prefetches for a long key
// range costs microseconds to issue and is partly dropped).
constexpr int ATT_PF = 3;
template <int HD>
__device__ __forceinline__ void attention_prefetch(const Ctx &c, const bf16 *kcache, const bf16 *vcache, size_t kv_lo, int lo,
                                                   int hi, int st) {
    constexpr int LPK = HD / 64;                         // 128-byte lines per key row
    if (st >= ((hi - lo + 7) >> 3)) return;
    for (int idx = c.lane; idx < 32 * LPK; idx += 32) {
        const int line = idx % LPK, key = (idx / LPK) & 7, plane = (idx / (LPK * 8)) & 1, tens = idx / (LPK * 16);
        const bf16 *ptr = (tens ? vcache : kcache) + plane * kv_lo + (size_t)min(lo + st * 8 + key, hi - 1) * HD + line * 64;
        asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
    }
}

// The key loop of one warp: keys in steps of 8 (step st, st + KW, ...), first the
// cached keys [lo, hi), then (last split only) the n_r keys of this forward, which
// row j sees up to key j (jrow: the sequence row of the lane's two query rows, -1 for
// an idle query row).  mt: the warp's 16-row query tile.  Leaves running max,
// sum (this lane's share) and un-normalised output of rows g and g+8 of the tile.
// Products of two remainders (2^-18 relative) are left out.
template <int HD, bool WIDE>
__device__ __forceinline__ void attention_keys(Ctx &c, const bf16 *kcache, const bf16 *vcache, size_t kv_lo, int lo, int hi,
                                               int n_new, int n_r, int fresh_lo, const int (&jrow)[2], int pos0, int mt, int kw,
                                               int KW, float (&mx)[2], float (&lsum)[2], float (&o)[HD / 8][4]) {
    using SM = AttSmem<HD>;
    constexpr int NCH = HD / 32, NOT = HD / 8, QP = SM::QP, VP = SM::VP;
    const int g = c.lane >> 2, t = c.lane & 3;
    const bf16 *kn = reinterpret_cast<const bf16 *>(c.scratch + SM::KN_OFF), *vn = reinterpret_cast<const bf16 *>(c.scratch + SM::VN_OFF);
    // With two query tiles, warps w and w + 4 walk the same key steps: warp w stages the V rows for both (they
    // meet at a named barrier of 64 threads before and after the P V products).
    const bool shared_v = KW == 4, loader = !shared_v || c.warp < 4;
    unsigned char *vslot = c.scratch + SM::VS_OFF + (shared_v ? (c.warp & 3) : c.warp) * (16 * VP);
    auto pair_sync = [&]() {
        if (shared_v) asm volatile("bar.sync %0, 64;" ::"r"(3 + (c.warp & 3)) : "memory");
    };
    const unsigned char *q0 = c.scratch + SM::Q_OFF + (mt * 16 + g) * QP + t * 16, *q1 = q0 + 8 * QP;
    const int steps_c = (hi - lo + 7) >> 3, steps_n = (n_new + 7) >> 3;
    for (int st = kw; st < steps_c + steps_n; st += KW) {
        const bool fresh = st >= steps_c;                // keys of this forward (from shared memory), else cached keys
        const int key0 = fresh ? (st - steps_c) * 8 : lo + st * 8;
        const int kend = fresh ? n_r : hi;               // first invalid key index
        const bf16 *kb = fresh ? kn : kcache, *vb = fresh ? vn : vcache;
        const size_t plane = fresh ? (size_t)32 * HD : kv_lo;
        // V of the step into this warp's slot: rows 0..7 the values of the 8 keys, rows 8..15 their remainders
        // (keys past the end repeat the last valid key: finite, and masked)
        for (int i = c.lane; loader && i < 16 * (HD / 8); i += 32) {
            const int kr = i / (HD / 8), piece = i - kr * (HD / 8);
            const bf16 *src = vb + (kr >> 3) * plane + (size_t)min(key0 + (kr & 7), kend - 1) * HD + piece * 8;
            if (fresh) *reinterpret_cast<uint4 *>(vslot + kr * VP + piece * 16) = *reinterpret_cast<const uint4 *>(src);
            else cp_async16(vslot + kr * VP + piece * 16, src);
        }
        if (hi > lo) attention_prefetch<HD>(c, kcache, vcache, kv_lo, lo, hi, st + ATT_PF * KW);
        // scores S = Q K^T for 8 keys: lane (g, t) reads 8 consecutive channels of key g and uses them as the
        // k slots {2t, 2t+1, 2t+8, 2t+9} of two MMAs; q is read with the same rule
        float s[4];
        {
            const bf16 *krow = kb + (size_t)min(key0 + g, kend - 1) * HD + t * 8;
            uint4 kf[NCH], kl[NCH];
#pragma unroll
            for (int cc = 0; cc < NCH; ++cc) {
                kf[cc] = *reinterpret_cast<const uint4 *>(krow + cc * 32);
                kl[cc] = *reinterpret_cast<const uint4 *>(krow + plane + cc * 32);
            }
            // two independent accumulators halve the chain of dependent MMAs (more of them spill registers)
            float sa[2][4];
#pragma unroll
            for (int e = 0; e < 2; ++e) sa[e][0] = sa[e][1] = sa[e][2] = sa[e][3] = 0.f;
#pragma unroll
            for (int cc = 0; cc < NCH; ++cc) {
                const uint4 qa = *reinterpret_cast<const uint4 *>(q0 + cc * 64), qb = *reinterpret_cast<const uint4 *>(q1 + cc * 64);
                mma16816(sa[0], qa.x, qb.x, qa.y, qb.y, kf[cc].x, kf[cc].y);
                mma16816(sa[1], qa.z, qb.z, qa.w, qb.w, kf[cc].z, kf[cc].w);
                mma16816(sa[0], qa.x, qb.x, qa.y, qb.y, kl[cc].x, kl[cc].y);
                mma16816(sa[1], qa.z, qb.z, qa.w, qb.w, kl[cc].z, kl[cc].w);
                const uint4 la = *reinterpret_cast<const uint4 *>(q0 + 32 * QP + cc * 64);
                const uint4 lb = *reinterpret_cast<const uint4 *>(q1 + 32 * QP + cc * 64);
                mma16816(sa[0], la.x, lb.x, la.y, lb.y, kf[cc].x, kf[cc].y);
                mma16816(sa[1], la.z, lb.z, la.w, lb.w, kf[cc].z, kf[cc].w);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) s[i] = sa[0][i] + sa[1][i];
        }
        // mask: keys past the end; among the keys of this forward, row j sees keys 0..j
        float rmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int key = key0 + 2 * t + (i & 1), row = jrow[i >> 1];      // row of the sequence this query row is
            // (with a restricted attention context the keys of this forward before fresh_lo are outside it;
            // a row always sees itself)
            // (WIDE: the new keys are in the cache too, key index = cache position: row j sees up to position pos0 + j)
            const bool ok = key < kend && (fresh ? (key <= row && (key >= fresh_lo || key == row)) : (!WIDE || key <= pos0 + row));
            if (!ok) s[i] = -INFINITY;
            rmax[i >> 1] = fmaxf(rmax[i >> 1], s[i]);
        }
        float corr[2];
#pragma unroll
        for (int hr = 0; hr < 2; ++hr) {
            rmax[hr] = fmaxf(rmax[hr], __shfl_xor_sync(0xffffffffu, rmax[hr], 1));
            rmax[hr] = fmaxf(rmax[hr], __shfl_xor_sync(0xffffffffu, rmax[hr], 2));
            const float mnew = fmaxf(mx[hr], rmax[hr]);
            corr[hr] = mnew == -INFINITY ? 1.f : __expf(mx[hr] - mnew);
            mx[hr] = mnew;
            lsum[hr] *= corr[hr];
        }
        uint32_t ph[2], pl[2];                           // probabilities of rows g / g+8, keys 2t, 2t+1: values, remainders
        {
            float p[4], r[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float mm = mx[i >> 1];
                p[i] = mm == -INFINITY ? 0.f : __expf(s[i] - mm);
                lsum[i >> 1] += p[i];
                r[i] = p[i] - __bfloat162float(__float2bfloat16(p[i]));
            }
            ph[0] = pack_bf16x2(p[0], p[1]); ph[1] = pack_bf16x2(p[2], p[3]);
            pl[0] = pack_bf16x2(r[0], r[1]); pl[1] = pack_bf16x2(r[2], r[3]);
        }
#pragma unroll
        for (int i = 0; i < NOT; ++i) { o[i][0] *= corr[0]; o[i][1] *= corr[0]; o[i][2] *= corr[1]; o[i][3] *= corr[1]; }
        // O += P V: V^T fragments through ldmatrix.trans from the slot.  Lane l gives the row address of
        // matrix l / 8: slot rows 0..7 or 8..15 (bit 3 of l), channel tile 0 or 1 of the pair (bit 4 of l).
        // The 16 k slots of an MMA are the 8 keys' values and then their remainders, so the probabilities
        // appear twice in the first product; the second adds (remainder of P) x (values of V).
        cp_async_wait_all();
        __syncwarp();
        pair_sync();                                     // the slot is filled, for both warps of a pair
        const unsigned char *vrow = vslot + ((c.lane & 7) + ((c.lane >> 3) & 1) * 8) * VP + (c.lane >> 4) * 16;
#pragma unroll
        for (int np = 0; np < NOT / 2; ++np) {
            uint32_t vf[4];
            ldmatrix_x4_trans(vf, vrow + np * 32);
            mma16816(o[2 * np], ph[0], ph[1], ph[0], ph[1], vf[0], vf[1]);
            mma16816(o[2 * np], pl[0], pl[1], 0u, 0u, vf[0], vf[1]);
            mma16816(o[2 * np + 1], ph[0], ph[1], ph[0], ph[1], vf[2], vf[3]);
            mma16816(o[2 * np + 1], pl[0], pl[1], 0u, 0u, vf[2], vf[3]);
        }
        __syncwarp();                                    // the slot is read; the next step may overwrite it
        pair_sync();
    }
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
        lsum[hr] += __shfl_xor_sync(0xffffffffu, lsum[hr], 1);
        lsum[hr] += __shfl_xor_sync(0xffffffffu, lsum[hr], 2);
    }
}

template <int HD, bool GQA, bool WIDE>
__device__ __forceinline__ void attention_item(Ctx &c, const Args &a, int layer, int seq, int kh, int vc, int split, int nsplit) {
    const XLay xl{a.g.nt, a.g.G};
    using SM = AttSmem<HD>;
    constexpr int PW = SM::PW, NOT = HD / 8;
    const DevPtrs &d = a.d;
    const ModelDev &m = a.m;
    const int H = m.cfg.n_heads, Hkv = m.cfg.n_kv_heads, group = GQA ? H / Hkv : 1;
    const int n_r = c.n_rows[seq], r_base = seq * a.g.rps, pos0 = c.row_pos[r_base];
    const int vbase = GQA ? 32 * vc : 0, nv = GQA ? min(32, group * n_r - vbase) : n_r;      // this item's virtual query rows
    const size_t cbase = (((size_t)layer * d.max_batch + seq) * Hkv + kh) * (size_t)d.max_ctx * HD;
    // cached keys in the attention context: [ks, pos0); WIDE: up to the last new row this item's query rows see
    int kv_end = pos0;
    if (WIDE) { const int v_last = vbase + nv - 1; kv_end = pos0 + 1 + (vbase / n_r != v_last / n_r ? n_r - 1 : v_last % n_r); }
    const int ks = min(c.key_start[seq], pos0), span = kv_end - ks;
    const int lo = ks + (int)((long long)span * split / nsplit), hi = ks + (int)((long long)span * (split + 1) / nsplit);
    const int fresh_lo = max(0, c.key_start[seq] - pos0);
    const int two = nv > 16 ? 1 : 0;                     // two query tiles: warps 0..3 take rows 0..15, warps 4..7 rows 16..31
    const int mt = two ? (c.warp >> 2) : 0, kw = two ? (c.warp & 3) : c.warp, KW = two ? 4 : 8;
    const int g = c.lane >> 2, t = c.lane & 3;
    int jrow[2];
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
        const int lv = mt * 16 + g + 8 * hr;
        jrow[hr] = GQA ? (lv < nv ? (vbase + lv) % n_r : -1) : lv;
    }
    if (hi > lo)
        for (int i = 0; i < ATT_PF; ++i) attention_prefetch<HD>(c, m.kcache + cbase, m.vcache + cbase, m.kv_lo, lo, hi, kw + i * KW);
    attention_rows<HD, GQA, !WIDE>(c, a, layer, seq, kh, vbase, nv, !WIDE && split == 0 && vc == 0);
    bsync();
    float mx[2] = {-INFINITY, -INFINITY}, lsum[2] = {0.f, 0.f};
    float o[NOT][4];
#pragma unroll
    for (int i = 0; i < NOT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    attention_keys<HD, WIDE>(c, m.kcache + cbase, m.vcache + cbase, m.kv_lo, lo, hi, (!WIDE && split == nsplit - 1) ? n_r : 0, n_r,
                             fresh_lo, jrow, pos0, mt, kw, KW, mx, lsum, o);

    bsync();                                             // every warp is done with q, the new rows and the slots
    float *red = reinterpret_cast<float *>(c.scratch);   // [8 warps][16 rows][PW]
    {
        float *rw0 = red + ((size_t)c.warp * 16 + g) * PW, *rw1 = rw0 + 8 * PW;
#pragma unroll
        for (int i = 0; i < NOT; ++i) {
            rw0[i * 8 + 2 * t] = o[i][0]; rw0[i * 8 + 2 * t + 1] = o[i][1];
            rw1[i * 8 + 2 * t] = o[i][2]; rw1[i * 8 + 2 * t + 1] = o[i][3];
        }
        if (t == 0) { rw0[HD] = mx[0]; rw0[HD + 1] = lsum[0]; rw1[HD] = mx[1]; rw1[HD + 1] = lsum[1]; }
    }
    bsync();
    // merge the warps of each query tile -> the item's partial in global memory; with a single split the
    // result is final and goes straight to the output projection's input buffer
    // per (row, warp) the factor exp(max_w - max) once, then one multiply-add per warp and output channel
    float *fw = red + MMA_WARPS * 16 * PW;               // [row][8] factors, then [row] max, [row] sum
    float *rowM = fw + 32 * MMA_WARPS, *rowL = rowM + 32;
    if (threadIdx.x < nv) {
        const int j = threadIdx.x, w0 = two ? (j >> 4) * 4 : 0, rr = j & 15;
        float M = -INFINITY;
        for (int w = 0; w < KW; ++w) M = fmaxf(M, red[((size_t)(w0 + w) * 16 + rr) * PW + HD]);
        float L = 0.f;
        for (int w = 0; w < KW; ++w) {
            const float *rw = red + ((size_t)(w0 + w) * 16 + rr) * PW;
            const float f = rw[HD] == -INFINITY ? 0.f : __expf(rw[HD] - M);
            fw[j * MMA_WARPS + w] = f;
            L += rw[HD + 1] * f;
        }
        rowM[j] = M; rowL[j] = L;
    }
    bsync();
    for (int i = threadIdx.x; i < nv * HD; i += MMA_THREADS) {
        const int lv = i / HD, ch = i - lv * HD;
        const int w0 = two ? (lv >> 4) * 4 : 0, rr = lv & 15;
        int h = kh, j = lv;                              // the head and sequence row this query row is
        if (GQA) { const int v = vbase + lv, hq = v / n_r; j = v - hq * n_r; h = kh * group + hq; }
        float ov = 0.f;
        for (int w = 0; w < KW; ++w) ov += red[((size_t)(w0 + w) * 16 + rr) * PW + ch] * fw[lv * MMA_WARPS + w];
        if (nsplit == 1) {
            store_split(d.att, xl, r_base + j, h * HD + ch, ov / rowL[lv]);
        } else {
            float *op = a.fb.attp + ((((size_t)(seq * H + h) * MAX_SPLIT + split) * a.g.rps) + j) * PW;
            op[ch] = ov;
            if (ch == 0) { op[HD] = rowM[lv]; op[HD + 1] = rowL[lv]; }
        }
    }
    bsync();
}

// Items of one (sequence, kv head) and key split: one per 32 virtual query rows (group * rows of the sequence).
__device__ __forceinline__ int attention_chunks(const Args &a) {
    const int group = a.m.cfg.n_heads / a.m.cfg.n_kv_heads;
    return (group == 1 && a.g.rps <= 32) ? 1 : (group * a.g.rps + 31) / 32;
}

// Key-range splits of a head in this forward (the same value in every block).  With fewer (sequence, head)
// pairs than blocks: as many splits as give every block at most one item.  With more pairs than blocks (batches
// with long contexts) the items take several rounds, and the number of splits is the one with the least
// rounds x (keys of an item + the fixed cost of an item, about 128 keys' worth).
__device__ __forceinline__ int attention_splits(const Ctx &c, const Args &a) {
    int lmax = 0;
    for (int s = 0; s < a.g.batch; ++s)
        if (c.n_rows[s] > 0) lmax = max(lmax, c.row_pos[s * a.g.rps] + (a.g.rps > 32 ? c.n_rows[s] : 0));
    const int pairs = a.g.batch * a.m.cfg.n_kv_heads * attention_chunks(a), cap = max(1, min(MAX_SPLIT, lmax / 64));
    if (pairs <= c.ncta) return max(1, min(c.ncta / pairs, cap));
    int best = 1;
    long long best_cost = -1;
    for (int n = 1; n <= cap; ++n) {
        const long long rounds = (pairs * n + c.ncta - 1) / c.ncta, cost = rounds * (lmax / n + 128);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = n; }
    }
    return best;
}

// All blocks, after the grid barrier that follows the items: the splits of every
// (sequence, head, row) merged by one warp each, into the bf16 attention output in
// the operand order the output projection reads.
__device__ __forceinline__ void phase_attention_merge(Ctx &c, const Args &a, int nsplit) {
    const XLay xl{a.g.nt, a.g.G};
    const int H = a.m.cfg.n_heads, hd = a.m.hd, PW = hd + 2, rps = a.g.rps;
    const int tasks = a.g.batch * H * rps;
    for (int task = c.cta * MMA_WARPS + c.warp; task < tasks; task += c.ncta * MMA_WARPS) {
        const int j = task % rps, sh = task / rps, h = sh % H, seq = sh / H;
        if (j >= c.n_rows[seq]) continue;
        const float *base = a.fb.attp + ((size_t)(seq * H + h) * MAX_SPLIT * rps + j) * PW;
        float M = -INFINITY;
        for (int sp = 0; sp < nsplit; ++sp) M = fmaxf(M, __ldcg(base + (size_t)sp * rps * PW + hd));
        float L = 0.f, ov[4] = {0.f, 0.f, 0.f, 0.f};
        for (int sp = 0; sp < nsplit; ++sp) {
            const float *pp = base + (size_t)sp * rps * PW;
            const float ms = __ldcg(pp + hd);
            const float f = ms == -INFINITY ? 0.f : __expf(ms - M);
            L += __ldcg(pp + hd + 1) * f;
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (c.lane + 32 * e < hd) ov[e] += __ldcg(pp + c.lane + 32 * e) * f;
        }
        const float inv = 1.f / L;
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (c.lane + 32 * e < hd)
                store_split(a.d.att, xl, seq * rps + j, h * hd + c.lane + 32 * e, ov[e] * inv);
    }
}

// All blocks: the attention items of one layer.  Forwards with more than 32 rows per sequence (prompt chunks) first
// append all new keys and values to the cache, pass a grid barrier, and then read every key from the cache.
__device__ __forceinline__ void phase_attention(Ctx &c, const Args &a, int layer, int nsplit) {
    const int Hkv = a.m.cfg.n_kv_heads, group = a.m.cfg.n_heads / Hkv, batch = a.g.batch, nvc = attention_chunks(a);
    const bool wide = a.g.rps > 32;
    if (wide) {
        const int nrc = (a.g.rps + 31) / 32, n_app = batch * Hkv * nrc;
        for (int it = c.cta; it < n_app; it += c.ncta) {
            const int jbase = (it % nrc) * 32, r1 = it / nrc, kh = r1 % Hkv, seq = r1 / Hkv;
            if (jbase >= c.n_rows[seq]) continue;
            if (a.m.hd == 64) attention_append<64>(c, a, layer, seq, kh, jbase);
            else attention_append<128>(c, a, layer, seq, kh, jbase);
        }
        grid_barrier(c, a.fb);
    }
    const int items = batch * Hkv * nvc * nsplit;
    for (int it = c.cta; it < items; it += c.ncta) {
        const int split = it % nsplit, r1 = it / nsplit, vc = r1 % nvc, r2 = r1 / nvc, kh = r2 % Hkv, seq = r2 / Hkv;
        if (c.n_rows[seq] == 0 || 32 * vc >= group * c.n_rows[seq]) continue;
        if (wide) {
            if (a.m.hd == 64) attention_item<64, true, true>(c, a, layer, seq, kh, vc, split, nsplit);
            else attention_item<128, true, true>(c, a, layer, seq, kh, vc, split, nsplit);
        } else if (group == 1) {
            if (a.m.hd == 64) attention_item<64, false, false>(c, a, layer, seq, kh, vc, split, nsplit);
            else attention_item<128, false, false>(c, a, layer, seq, kh, vc, split, nsplit);
        } else {
            if (a.m.hd == 64) attention_item<64, true, false>(c, a, layer, seq, kh, vc, split, nsplit);
            else attention_item<128, true, false>(c, a, layer, seq, kh, vc, split, nsplit);
        }
    }
}

}  // namespace fwd
