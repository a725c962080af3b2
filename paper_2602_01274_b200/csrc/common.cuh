// Shared definitions of the Pacer CUDA library (device state, row geometry,
// activation layout of the standalone GEMM).  sm_100a only.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/pacer.h"

typedef __nv_bfloat16 bf16;

// Per-sequence decoding state, resident on the device.  Every kernel derives its
// row counts and positions from this, so no host decision is needed per step.
struct SeqState {
    int32_t P;            // accepted tokens so far (prompt included)
    int32_t len_T, len_D, len_B;
    int32_t gamma;        // drafts made in this step
    int32_t k_round;      // blocks that passed in this step
    float t_k;            // current threshold
    int32_t drafting;
    int32_t finished;
    int32_t n_steps;
    int32_t last_n, last_next;
    int32_t n_pend;       // hidden rows queued for M_B
    int32_t err;
    int32_t n_prompt, max_new;
    int64_t n_draft_fwd, n_mb_calls, n_target_fwd;
    int32_t gamma_max;    // window cap of this run (multiple of b)
    float t0;             // initial threshold, < 0: always pass
    int32_t mode;         // PACER_GREEDY / PACER_SAMPLE
    int32_t active;       // 1 for sequences 0..batch-1 of the current run
    uint64_t seed;
    int32_t mb_start;     // M_B cache position of the first draft row of this step (local-draft attention context)
    int32_t sched;        // 1: the window of every step is prescribed (no pre-verification), see DevPtrs::sched_win
    int32_t n_sched;      // prescribed windows per sequence (steps beyond reuse the last one)
    int32_t pad_;
};

enum RowKind {
    KIND_DRAFT = 0,      // rows of one draft forward (1, or 2 when catching up)
    KIND_VERIFY = 1,     // [last accepted, y_1..y_gamma]
    KIND_AR = 2,         // one row: the last accepted token
    KIND_PREFILL = 3,    // prompt rows c0..c0+rps-1 by token id
    KIND_MB = 4,         // hidden rows queued for the pre-verification model
    KIND_PREFILL_B = 5   // draft hidden rows of a prefill chunk, for M_B
};

// Row geometry of a forward: row r = seq * rps + j.  For the tensor cores the rows form G groups of nt
// eight-row tiles (a group's values and rounding remainders together fill at most the 128 rows of one MMA).
struct Geom {
    int32_t batch, rps, rtot;
    int32_t nt;                     // eight-row tiles per group: 1..4, 6 or 8
    int32_t G;                      // groups: 1, or up to 3 when nt is 6 or 8
    int32_t rpad;                   // G * nt * 8 >= rtot
};

// Device addresses of everything a kernel may need, passed by value.
struct DevPtrs {
    SeqState *st;
    int32_t *x;          // [max_batch][max_ctx] accepted tokens
    int32_t *y;          // [max_batch][gamma_cap] drafts of the current step
    float *alpha;        // [max_batch][gamma_cap]
    float *hpend;        // [max_batch][b+1][d_D]
    int32_t *hpend_e;    // [max_batch][b+1] draft index (1-based) or 0 for history rows
    int32_t *draft_len;  // [max_batch][max_steps]
    int32_t *accept_len; // [max_batch][max_steps]
    int32_t *sched_win;  // [max_batch][max_steps] prescribed windows (runs with SeqState::sched)
    int32_t sched_rows;  // rows per sequence of a draft forward in such a run (the draft may have rows to catch up on)
    float *verify_logits;// [max_batch][gamma_cap+1][V]
    float *draft_logits; // [max_batch][gamma_cap][V]
    // per-forward scratch
    int32_t *row_pos;    // [rtot] cache position of row r, -1 = inactive
    int32_t *row_tok;    // [rtot] input token (or draft index for M_B rows)
    int32_t *n_rows;     // [max_batch] active rows per sequence in this forward
    int32_t *row_arg;    // [rtot] argmax of the LM-head row
    float *row_margin;   // [rtot] top1 - top2
    float *xres;         // [rtot][d] fp32 residual stream
    bf16 *att;           // attention output, split bf16 in tensor-core operand order (K = H*hd)
    bf16 *act;           // SwiGLU output, split bf16 in tensor-core operand order (K = F)
    float *hidden;       // [rtot][d] fp32 final-norm output
    float *part;         // split-K partial sums [S][nt*8][N]
    int32_t max_batch, max_ctx, gamma_cap, block_b, max_steps;
    float rho, succ_bias;
    int32_t criterion, use_posemb, mb_scope;
};

struct ModelDev {
    pacer_model_cfg cfg;
    int32_t hd, qrows;
    const bf16 *embed, *wqkv, *wo, *wgate, *wup, *wdown, *norm1, *norm2, *normf, *head, *head_b, *posemb;
    const bf16 *wt[5];         // the five projections re-laid for the tensor cores (index: OpKind of the forward kernel)
    const int32_t *succ;
    bf16 *kcache, *vcache;     // [2][L][max_batch][Hkv][max_ctx][hd]: the bf16 values, then their rounding remainders
    size_t kv_lo;              // elements between the two parts
    const float2 *rope;        // [max_ctx][hd/2] (cos, sin)
    int32_t loaded;
};

// Offset (in elements) of X[r][k] in the fragment-major layout the standalone GEMM (pacer_linear) reads:
// [k/32][row tile][lane = (r%8)*4 + (k%32)/8][k%8].  A warp's 128-bit loads of
// one (32-wide k chunk, row tile) are 512 contiguous bytes, already in the
// register order of mma.m16n8k16's B operand (with the k permutation the GEMM
// applies to its A operand too).
__host__ __device__ __forceinline__ size_t xfrag_index(int r, int k, int nt_total) {
    return ((((size_t)(k >> 5) * nt_total + (r >> 3)) * 32 + ((r & 7) << 2) + ((k & 31) >> 3)) << 3) + (k & 7);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the block; every thread gets the result.  `red` is 33 floats of shared memory.
__device__ __forceinline__ float block_sum(float v, float *red) {
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    if (w == 0) {
        float t = lane < nw ? red[lane] : 0.f;
        t = warp_sum(t);
        if (lane == 0) red[32] = t;
    }
    __syncthreads();
    return red[32];
}
