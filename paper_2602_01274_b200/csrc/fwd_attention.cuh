// Attention phase of the forward kernel: rotary embedding of the new q/k rows,
// append of k/v to the bf16 cache, and causal attention of the new rows over the
// cache.  Work items are (sequence, head, key-range split); every item leaves an
// un-normalised partial (running max, sum, weighted values) and the item that
// finishes last for a (sequence, head) merges the splits and writes the bf16
// attention output in the fragment order the output projection reads.
#pragma once
#include "fwd_phases.cuh"

namespace fwd {

constexpr int ATT_RB = 8;      // query rows handled together by a warp
constexpr int ATT_WARPS = MMA_WARPS;

template <int EPL>             // channels per lane: hd = 32 * EPL
__device__ __forceinline__ void load_kv_row(const bf16 *p, float (&out)[EPL]) {
    if constexpr (EPL == 4) {
        const uint2 raw = *reinterpret_cast<const uint2 *>(p);
        const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
        const float2 a = __bfloat1622float2(h2[0]), b = __bfloat1622float2(h2[1]);
        out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
    } else if constexpr (EPL == 2) {
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(p));
        out[0] = a.x; out[1] = a.y;
    } else {
        out[0] = __bfloat162float(p[0]);
    }
}

template <int EPL>
__device__ __forceinline__ void attention_item(Ctx &c, const Args &a, int layer, int seq, int h, int split, int nsplit,
                                               int nt_total) {
    constexpr int hd = 32 * EPL, half = hd / 2, PW = hd + 2;
    const DevPtrs &d = a.d;
    const ModelDev &m = a.m;
    const int H = m.cfg.n_heads, Hkv = m.cfg.n_kv_heads, group = H / Hkv, kh = h / group, qrows = m.qrows;
    const int n_r = c.n_rows[seq], r_base = seq * a.g.rps;
    const int pos0 = c.row_pos[r_base];
    float *qs = reinterpret_cast<float *>(c.scratch);                       // [MAX_ROWS][hd]
    bf16 *kn = reinterpret_cast<bf16 *>(qs + MAX_ROWS * hd);                // [MAX_ROWS][hd]
    bf16 *vn = kn + MAX_ROWS * hd;
    float *red = reinterpret_cast<float *>(vn + MAX_ROWS * hd);             // [ATT_WARPS][ATT_RB][PW]
    const size_t cbase = (((size_t)layer * d.max_batch + seq) * Hkv + kh) * (size_t)d.max_ctx * hd;
    const bool writer = split == 0 && h == kh * group;
    const float scale = rsqrtf((float)hd);

    // rotary embedding of the new rows (rotate-half pairs (i, i + hd/2)); k and v rounded to bf16 as cached
    for (int i = threadIdx.x; i < n_r * half; i += MMA_THREADS) {
        const int j = i / half, ii = i - j * half, pos = pos0 + j;
        const float *row = a.fb.qkv + (size_t)(r_base + j) * qrows;
        const float2 cs = m.rope[(size_t)pos * half + ii];
        const float qa = __ldcg(row + h * hd + ii), qb = __ldcg(row + h * hd + ii + half);
        qs[j * hd + ii] = (qa * cs.x - qb * cs.y) * scale;
        qs[j * hd + ii + half] = (qb * cs.x + qa * cs.y) * scale;
        const float ka = __ldcg(row + (H + kh) * hd + ii), kb = __ldcg(row + (H + kh) * hd + ii + half);
        const bf16 k0 = __float2bfloat16(ka * cs.x - kb * cs.y), k1 = __float2bfloat16(kb * cs.x + ka * cs.y);
        const bf16 v0 = __float2bfloat16(__ldcg(row + (H + Hkv + kh) * hd + ii));
        const bf16 v1 = __float2bfloat16(__ldcg(row + (H + Hkv + kh) * hd + ii + half));
        kn[j * hd + ii] = k0; kn[j * hd + ii + half] = k1;
        vn[j * hd + ii] = v0; vn[j * hd + ii + half] = v1;
        if (writer) {
            bf16 *kc = m.kcache + cbase + (size_t)pos * hd, *vc = m.vcache + cbase + (size_t)pos * hd;
            kc[ii] = k0; kc[ii + half] = k1;
            vc[ii] = v0; vc[ii + half] = v1;
        }
    }
    bsync();

    const int lo = (int)((long long)pos0 * split / nsplit), hi = (int)((long long)pos0 * (split + 1) / nsplit);
    const bool with_new = split == nsplit - 1;
    const bf16 *kc = m.kcache + cbase + c.lane * EPL, *vc = m.vcache + cbase + c.lane * EPL;
    float *outp = a.fb.attp + (((size_t)(seq * H + h) * MAX_SPLIT + split) * a.g.rps) * PW;

    for (int j0 = 0; j0 < n_r; j0 += ATT_RB) {
        const int nrb = min(ATT_RB, n_r - j0);
        float mx[ATT_RB], den[ATT_RB], acc[ATT_RB][EPL], qv[ATT_RB][EPL];
#pragma unroll
        for (int jj = 0; jj < ATT_RB; ++jj) {
            mx[jj] = -INFINITY; den[jj] = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                acc[jj][e] = 0.f;
                qv[jj][e] = jj < nrb ? qs[(j0 + jj) * hd + c.lane * EPL + e] : 0.f;
            }
        }
        auto one_key = [&](const float (&kk)[EPL], const float (&vv)[EPL], int first_row) {
#pragma unroll
            for (int jj = 0; jj < ATT_RB; ++jj) {
                if (jj < nrb && j0 + jj >= first_row) {
                    float sc = 0.f;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) sc += qv[jj][e] * kk[e];
                    sc = warp_sum(sc);
                    const float mnew = fmaxf(mx[jj], sc);
                    const float corr = __expf(mx[jj] - mnew), w = __expf(sc - mnew);
                    den[jj] = den[jj] * corr + w;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) acc[jj][e] = acc[jj][e] * corr + w * vv[e];
                    mx[jj] = mnew;
                }
            }
        };
        const bool walker = true;
        for (int p = lo + c.warp; walker && p < hi; p += ATT_WARPS) {   // cached keys: every new row sees them
            float kk[EPL], vv[EPL];
            load_kv_row<EPL>(kc + (size_t)p * hd, kk);
            load_kv_row<EPL>(vc + (size_t)p * hd, vv);
            one_key(kk, vv, 0);
        }
        if (with_new && walker) {                                // new keys: row j sees new keys 0..j
            for (int jn = c.warp; jn < n_r; jn += ATT_WARPS) {
                float kk[EPL], vv[EPL];
                load_kv_row<EPL>(kn + jn * hd + c.lane * EPL, kk);
                load_kv_row<EPL>(vn + jn * hd + c.lane * EPL, vv);
                one_key(kk, vv, jn);
            }
        }
        // merge the warps' partials of this row block
#pragma unroll
        for (int jj = 0; walker && jj < ATT_RB; ++jj) {
            float *rw = red + ((size_t)c.warp * ATT_RB + jj) * PW;
#pragma unroll
            for (int e = 0; e < EPL; ++e) rw[c.lane * EPL + e] = acc[jj][e];
            if (c.lane == 0) { rw[hd] = mx[jj]; rw[hd + 1] = den[jj]; }
        }
        bsync();
        for (int i = threadIdx.x; i < nrb * hd; i += MMA_THREADS) {
            const int jj = i / hd, ch = i - jj * hd;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < ATT_WARPS; ++w) M = fmaxf(M, red[((size_t)w * ATT_RB + jj) * PW + hd]);
            float L = 0.f, o = 0.f;
#pragma unroll
            for (int w = 0; w < ATT_WARPS; ++w) {
                const float *rw = red + ((size_t)w * ATT_RB + jj) * PW;
                const float f = rw[hd] == -INFINITY ? 0.f : __expf(rw[hd] - M);
                L += rw[hd + 1] * f;
                o += rw[ch] * f;
            }
            float *op = outp + (size_t)(j0 + jj) * PW;
            op[ch] = o;
            if (ch == 0) { op[hd] = M; op[hd + 1] = L; }
        }
        bsync();
    }

    // the item that finishes last for (seq, h) merges the splits
    __threadfence();
    bsync();
    if (threadIdx.x == 0) {
        const int old = atomicAdd(a.fb.att_cnt + seq * H + h, 1);
        c.flag[0] = old == nsplit - 1;
        if (old == nsplit - 1) a.fb.att_cnt[seq * H + h] = 0;
    }
    bsync();
    if (c.flag[0]) {
        __threadfence();
        const float *base = a.fb.attp + ((size_t)(seq * H + h) * MAX_SPLIT) * a.g.rps * PW;
        for (int i = threadIdx.x; i < n_r * hd; i += MMA_THREADS) {
            const int j = i / hd, ch = i - j * hd;
            float M = -INFINITY;
            for (int sp = 0; sp < nsplit; ++sp) M = fmaxf(M, __ldcg(base + ((size_t)sp * a.g.rps + j) * PW + hd));
            float L = 0.f, o = 0.f;
            for (int sp = 0; sp < nsplit; ++sp) {
                const float *pp = base + ((size_t)sp * a.g.rps + j) * PW;
                const float ms = __ldcg(pp + hd);
                const float f = ms == -INFINITY ? 0.f : __expf(ms - M);
                L += __ldcg(pp + hd + 1) * f;
                o += __ldcg(pp + ch) * f;
            }
            d.att[xfrag_index(r_base + j, h * hd + ch, nt_total)] = __float2bfloat16(o / L);
        }
    }
    bsync();
}

// All blocks: the attention of one layer.
__device__ __forceinline__ void phase_attention(Ctx &c, const Args &a, int layer, int nt_total) {
    const int H = a.m.cfg.n_heads, batch = a.g.batch;
    int lmax = 0;
    for (int s = 0; s < batch; ++s)
        if (c.n_rows[s] > 0) lmax = max(lmax, c.row_pos[s * a.g.rps]);
    int nsplit = c.ncta / (batch * H);
    nsplit = max(1, min(nsplit, min(MAX_SPLIT, lmax / 64)));
    const int items = batch * H * nsplit;
    for (int it = c.cta; it < items; it += c.ncta) {
        const int split = it % nsplit, sh = it / nsplit, h = sh % H, seq = sh / H;
        if (c.n_rows[seq] == 0) continue;
        switch (a.m.hd) {
            case 32: attention_item<1>(c, a, layer, seq, h, split, nsplit, nt_total); break;
            case 64: attention_item<2>(c, a, layer, seq, h, split, nsplit, nt_total); break;
            default: attention_item<4>(c, a, layer, seq, h, split, nsplit, nt_total); break;
        }
    }
}

}  // namespace fwd
