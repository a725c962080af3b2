// Skinny weight-streaming GEMM: Y[r][n] = sum_k X[r][k] * W[n][k], rows <= 32.
//
// The path is bound by reading W once from HBM, so the kernel is organised
// around that stream: every lane reads its share of W with 128-bit loads straight
// into registers (each weight is used exactly once, so staging it in shared
// memory would only add traffic), several loads in flight per lane.  The few
// activation rows sit in shared memory in fragment order.  Tensor cores
// (mma.m16n8k16, bf16 in, fp32 accumulate) do the contraction with the WEIGHTS
// as the 16-row operand and the token rows as the 8-wide operand, so 1..4 row
// tiles cost 2..8 MMAs per KB of weights and the math stays invisible.
//
// k permutation: inside every 32-wide k chunk a lane (g = lane/4, t = lane%4)
// loads the 8 consecutive weights W[n][32c + 8t .. 8t+7] and uses them as the k
// slots {2t,2t+1,2t+8,2t+9} of two MMAs.  The activation fragment is loaded with
// the same rule, so the products pair up correctly and the sum over k is the same.
//
// Split-K: the grid is S k-slices x row-tile groups; slice partial sums go to
// part[slice][row][n] and are added up, in slice order (deterministic), by the
// kernel that consumes the result.
#pragma once
#include "common.cuh"

__device__ __forceinline__ uint4 ldg_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct GemmArgs {
    const bf16 *X;       // fragment-major activations
    int32_t nt_total;    // row tiles in X's layout
    int32_t nt_off;      // first row tile this launch covers
    const bf16 *W1;      // rows [0, n_w1)
    const bf16 *W2;      // rows [n_w1, N) (e.g. gate rows then up rows), or unused
    int32_t n_w1;
    int32_t N, K;
    int32_t KS;          // k-slice length, multiple of 32
    int32_t S;           // number of k slices
    int32_t tpw;         // weight-row tiles (16 rows) per warp
    float *part;         // [S][rpad][N]
    int32_t rpad;        // rows stride of part (= nt_total * 8)
    const int32_t *n_rows; // per-sequence active rows of this forward; NULL = always run
    int32_t n_seq;
};

constexpr int GEMM_THREADS = 256;
constexpr int GEMM_PF = 6;       // 128-bit weight loads in flight per lane and row half

template <int NT>
__global__ void __launch_bounds__(GEMM_THREADS) k_gemm_skinny(const GemmArgs a) {
    extern __shared__ uint4 xs[];                      // [chunks][NT][32] 16-byte fragments
    if (a.n_rows) {                                    // nothing to do when every sequence idles
        int any = 0;
        for (int s = 0; s < a.n_seq; ++s) any |= a.n_rows[s];
        if (!any) return;
    }
    const int slice = blockIdx.x % a.S, grp = blockIdx.x / a.S;
    const int k0 = slice * a.KS;
    const int kend = min(a.K, k0 + a.KS);
    const int nchunks = (kend - k0) >> 5;
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(a.X);
        const int per_chunk = NT * 32;
        for (int i = threadIdx.x; i < nchunks * per_chunk; i += GEMM_THREADS) {
            int c = i / per_chunk, rem = i - c * per_chunk;
            xs[i] = src[((size_t)((k0 >> 5) + c) * a.nt_total + a.nt_off) * 32 + rem];
        }
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int MT = (a.N + 15) >> 4;
    const int mt_first = grp * a.tpw * 8 + warp;       // this warp's tiles: mt_first + 8*i
    int ntile_w = 0;
    for (int i = 0; i < a.tpw; ++i) if (mt_first + 8 * i < MT) ntile_w = i + 1;
    if (ntile_w == 0) return;
    const int total = ntile_w * nchunks;               // flat (tile, chunk) sequence of this warp

    auto row_ptr = [&](int n) -> const bf16 * {
        n = min(n, a.N - 1);
        return (n < a.n_w1 ? a.W1 + (size_t)n * a.K : a.W2 + (size_t)(n - a.n_w1) * a.K) + k0 + 8 * t;
    };

    uint4 w0[GEMM_PF], w1[GEMM_PF];
    // loader cursor
    int l_tile = 0, l_chunk = 0;
    const bf16 *lp0 = row_ptr(mt_first * 16 + g), *lp1 = row_ptr(mt_first * 16 + g + 8);
    auto issue = [&](int slot) {
        w0[slot] = ldg_stream(lp0 + (l_chunk << 5));
        w1[slot] = ldg_stream(lp1 + (l_chunk << 5));
        if (++l_chunk == nchunks) {
            l_chunk = 0;
            ++l_tile;
            int mt = mt_first + 8 * l_tile;
            lp0 = row_ptr(mt * 16 + g);
            lp1 = row_ptr(mt * 16 + g + 8);
        }
    };
#pragma unroll
    for (int j = 0; j < GEMM_PF; ++j) if (j < total) issue(j);

    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f; }
    int c_tile = 0, c_chunk = 0;
    for (int q0 = 0; q0 < total; q0 += GEMM_PF) {
#pragma unroll
        for (int j = 0; j < GEMM_PF; ++j) {
            const int q = q0 + j;
            if (q < total) {
                const uint4 a0 = w0[j], a1 = w1[j];
                if (q + GEMM_PF < total) issue(j);
                const uint4 *xb = xs + (size_t)c_chunk * (NT * 32) + lane;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const uint4 b = xb[nt * 32];
                    mma_bf16_16816(acc[nt], a0.x, a1.x, a0.y, a1.y, b.x, b.y);
                    mma_bf16_16816(acc[nt], a0.z, a1.z, a0.w, a1.w, b.z, b.w);
                }
                if (++c_chunk == nchunks) {
                    // tile finished: accumulator (g, 2t..2t+1) = weight row n0+g x token rows 2t, 2t+1
                    const int n0 = (mt_first + 8 * c_tile) * 16 + g, n1 = n0 + 8;
                    float *pbase = a.part + (size_t)slice * a.rpad * a.N;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const int r0 = (a.nt_off + nt) * 8 + 2 * t;
                        if (n0 < a.N) {
                            pbase[(size_t)r0 * a.N + n0] = acc[nt][0];
                            pbase[(size_t)(r0 + 1) * a.N + n0] = acc[nt][1];
                        }
                        if (n1 < a.N) {
                            pbase[(size_t)r0 * a.N + n1] = acc[nt][2];
                            pbase[(size_t)(r0 + 1) * a.N + n1] = acc[nt][3];
                        }
                        acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
                    }
                    c_chunk = 0;
                    ++c_tile;
                }
            }
        }
    }
}

// Launch plan for one product.
struct GemmPlan {
    int S, KS, tpw, grid;
    size_t smem;
};

static inline GemmPlan gemm_plan(int N, int K, int NT) {
    GemmPlan p;
    const int MT = (N + 15) / 16;
    int ks_target = MT >= 1024 ? 2048 : 1024;
    // shared memory: NT * 8 rows * KS * 2 bytes, keep two blocks per SM possible
    while ((size_t)NT * 8 * ks_target * 2 > 96 * 1024) ks_target /= 2;
    p.S = (K + ks_target - 1) / ks_target;
    p.KS = (((K + p.S - 1) / p.S) + 31) / 32 * 32;
    p.S = (K + p.KS - 1) / p.KS;
    long tasks = (long)MT * p.S;
    long tpw = tasks / (8L * 2 * 148);
    if (tpw < 1) tpw = 1;
    if (tpw > 8) tpw = 8;
    p.tpw = (int)tpw;
    int groups = (MT + 8 * p.tpw - 1) / (8 * p.tpw);
    p.grid = groups * p.S;
    p.smem = (size_t)NT * 8 * p.KS * 2;
    return p;
}

template <int NT>
static cudaError_t gemm_launch_nt(const GemmArgs &a, const GemmPlan &p, cudaStream_t st) {
    static bool attr_set[64] = {};           // the opt-in is per device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(k_gemm_skinny<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    k_gemm_skinny<NT><<<p.grid, GEMM_THREADS, p.smem, st>>>(a);
    return cudaGetLastError();
}

// Y partials for all `nt_total` row tiles: passes of up to 4 tiles each.
// Returns the number of kernels launched through *launches.
static cudaError_t gemm_run(const bf16 *X, int nt_total, const bf16 *W1, const bf16 *W2, int n_w1, int N, int K,
                            float *part, const int32_t *n_rows, int n_seq, cudaStream_t st, GemmPlan *plan_out,
                            int64_t *launches) {
    const int NT = nt_total < 4 ? nt_total : 4;
    GemmPlan p = gemm_plan(N, K, NT);
    if (plan_out) *plan_out = p;
    for (int off = 0; off < nt_total; off += 4) {
        int nt = nt_total - off < 4 ? nt_total - off : 4;
        GemmArgs a;
        a.X = X; a.nt_total = nt_total; a.nt_off = off; a.W1 = W1; a.W2 = W2 ? W2 : W1; a.n_w1 = W2 ? n_w1 : N;
        a.N = N; a.K = K; a.KS = p.KS; a.S = p.S; a.tpw = p.tpw; a.part = part; a.rpad = nt_total * 8;
        a.n_rows = n_rows; a.n_seq = n_seq;
        GemmPlan pp = p;
        pp.smem = (size_t)nt * 8 * p.KS * 2;
        cudaError_t e;
        switch (nt) {
            case 1: e = gemm_launch_nt<1>(a, pp, st); break;
            case 2: e = gemm_launch_nt<2>(a, pp, st); break;
            case 3: e = gemm_launch_nt<3>(a, pp, st); break;
            default: e = gemm_launch_nt<4>(a, pp, st); break;
        }
        if (e != cudaSuccess) return e;
        if (launches) ++*launches;
    }
    return cudaSuccess;
}
