// Causal decode attention of the new rows of a forward against the bf16 KV cache.
// One block per (head, row): the row at cache position pos attends to keys
// 0..pos of its sequence (its own freshly appended key included).  Keys are
// split over the warps of the block, each lane owns hd/32 consecutive channels,
// scores are reduced with warp shuffles, softmax is online (running max and sum
// in fp32), and the warps' partial results are merged through shared memory.
#pragma once
#include "common.cuh"

constexpr int ATT_WARPS = 4;

template <int EPL>   // channels per lane: hd = 32 * EPL
__global__ void __launch_bounds__(ATT_WARPS * 32) k_attention(DevPtrs d, ModelDev m, Geom g, int layer) {
    const int h = blockIdx.x, r = blockIdx.y;
    const int pos = d.row_pos[r];
    if (pos < 0) return;
    const int s = r / g.rps;
    constexpr int hd = 32 * EPL;
    const int H = m.cfg.n_heads, Hkv = m.cfg.n_kv_heads, kh = h / (H / Hkv);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float scale = rsqrtf((float)hd);
    float qv[EPL];
    {
        const float *q = d.q + (size_t)r * H * hd + h * hd + lane * EPL;
#pragma unroll
        for (int e = 0; e < EPL; ++e) qv[e] = q[e] * scale;
    }
    const size_t base = (((size_t)layer * d.max_batch + s) * Hkv + kh) * d.max_ctx * hd;
    const bf16 *kc = m.kcache + base + lane * EPL, *vc = m.vcache + base + lane * EPL;
    float mx = -INFINITY, den = 0.f, acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    for (int p = warp; p <= pos; p += ATT_WARPS) {
        float kk[EPL], vv[EPL];
        if constexpr (EPL == 4) {
            const uint2 kr = *reinterpret_cast<const uint2 *>(kc + (size_t)p * hd);
            const uint2 vr = *reinterpret_cast<const uint2 *>(vc + (size_t)p * hd);
            const __nv_bfloat162 *k2 = reinterpret_cast<const __nv_bfloat162 *>(&kr);
            const __nv_bfloat162 *v2 = reinterpret_cast<const __nv_bfloat162 *>(&vr);
            float2 a = __bfloat1622float2(k2[0]), b = __bfloat1622float2(k2[1]);
            kk[0] = a.x; kk[1] = a.y; kk[2] = b.x; kk[3] = b.y;
            a = __bfloat1622float2(v2[0]); b = __bfloat1622float2(v2[1]);
            vv[0] = a.x; vv[1] = a.y; vv[2] = b.x; vv[3] = b.y;
        } else if constexpr (EPL == 2) {
            const __nv_bfloat162 k2 = *reinterpret_cast<const __nv_bfloat162 *>(kc + (size_t)p * hd);
            const __nv_bfloat162 v2 = *reinterpret_cast<const __nv_bfloat162 *>(vc + (size_t)p * hd);
            float2 a = __bfloat1622float2(k2), b = __bfloat1622float2(v2);
            kk[0] = a.x; kk[1] = a.y; vv[0] = b.x; vv[1] = b.y;
        } else {
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                kk[e] = __bfloat162float(kc[(size_t)p * hd + e]);
                vv[e] = __bfloat162float(vc[(size_t)p * hd + e]);
            }
        }
        float sc = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) sc += qv[e] * kk[e];
        sc = warp_sum(sc);
        const float mnew = fmaxf(mx, sc);
        const float corr = __expf(mx - mnew), w = __expf(sc - mnew);
        den = den * corr + w;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = acc[e] * corr + w * vv[e];
        mx = mnew;
    }
    __shared__ float sm_m[ATT_WARPS], sm_l[ATT_WARPS], sm_o[ATT_WARPS][hd];
    if (lane == 0) { sm_m[warp] = mx; sm_l[warp] = den; }
#pragma unroll
    for (int e = 0; e < EPL; ++e) sm_o[warp][lane * EPL + e] = acc[e];
    __syncthreads();
    if (warp == 0) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < ATT_WARPS; ++w) M = fmaxf(M, sm_m[w]);
        float L = 0.f, o[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[e] = 0.f;
#pragma unroll
        for (int w = 0; w < ATT_WARPS; ++w) {
            const float f = sm_m[w] == -INFINITY ? 0.f : __expf(sm_m[w] - M);
            L += sm_l[w] * f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) o[e] += sm_o[w][lane * EPL + e] * f;
        }
        const float inv = 1.f / L;
#pragma unroll
        for (int e = 0; e < EPL; ++e)
            d.att[xfrag_index(r, h * hd + lane * EPL + e, g.nt)] = __float2bfloat16(o[e] * inv);
    }
}

static cudaError_t attention_launch(const DevPtrs &d, const ModelDev &m, const Geom &g, int layer, cudaStream_t st) {
    dim3 grid(m.cfg.n_heads, g.rtot);
    switch (m.hd) {
        case 32: k_attention<1><<<grid, ATT_WARPS * 32, 0, st>>>(d, m, g, layer); break;
        case 64: k_attention<2><<<grid, ATT_WARPS * 32, 0, st>>>(d, m, g, layer); break;
        case 128: k_attention<4><<<grid, ATT_WARPS * 32, 0, st>>>(d, m, g, layer); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}
