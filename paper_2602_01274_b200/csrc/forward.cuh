// One decoder forward as ONE persistent cooperative kernel (one block per SM).
//
// The forward is bound by streaming the weights from HBM once, so the kernel is
// built around an uninterrupted weight stream:
//   - every warp owns a private pipeline of shared-memory stages that it fills
//     itself with bulk async copies (cp.async.bulk + mbarrier) of 16 weight rows
//     x 256 k each; the list of (projection, tile, k-range) units a warp will
//     need is static, so a warp keeps issuing copies for the NEXT projection
//     while the block sits in a grid barrier or in a small phase (attention,
//     tail): the HBM queue never drains between projections;
//   - the few activation rows of a projection live in shared memory in MMA
//     fragment order; tensor cores (mma.m16n8k16, bf16 in / fp32 accumulate,
//     weights as the 16-row operand) do the contraction, so the math is invisible;
//   - a projection is cut into (k-slice, column-group) items spread over the
//     blocks; the warp that delivers the last k-slice of a 16-column tile sums
//     the slices in slice order (deterministic) and applies the row-wise step
//     that follows the projection in the decoder (residual add + RMS statistics,
//     SwiGLU, bias/arg-max of the LM head), so no separate row kernels exist;
//   - the streaming warps never wait on global-memory round trips: each hands
//     its finished accumulators through shared memory to a partner "epilogue"
//     warp, which does the stores, fences, arrival counting and row-wise steps;
//   - phases are separated by grid barriers with bounded waits.
#pragma once
#include "common.cuh"

namespace fwd {

constexpr int THREADS = 512, WARPS = 16;         // warps 0..7 stream weights and do the MMAs, warps 8..15 are their epilogue partners
constexpr int MMA_WARPS = 8;
constexpr int KC = 256;                         // k columns of one weight unit
constexpr int PITCH = KC * 2 + 64;              // bytes between the rows of a stage (bank-conflict free)
constexpr int STAGE_BYTES = 16 * PITCH;         // 9216
constexpr int STAGES = 2;
constexpr int RING_BYTES = MMA_WARPS * STAGES * STAGE_BYTES;   // 147456
constexpr int XBUF_BYTES = 64 * 1024;           // activation slice of a projection item
constexpr int HAND_BYTES = MMA_WARPS * 2048;    // accumulator hand-over buffers (4 row tiles x 4 x 32 lanes x fp32 each)
constexpr int SCRATCH_BYTES = XBUF_BYTES + HAND_BYTES;   // the attention phase and the tails use both, contiguously
constexpr int MISC_BYTES = 2048;
constexpr int SMEM_BYTES = SCRATCH_BYTES + RING_BYTES + MISC_BYTES;
constexpr int MAX_ROWS = 32;                    // rows of one forward (all sequences together)
constexpr int MAX_SPLIT = 16;                   // key-range splits of one attention head
constexpr unsigned SPIN_LIMIT = 1u << 22;
constexpr int PROF_STAMPS = 512;              // phase-boundary time stamps kept per block and forward
constexpr int PROF_BLOCKS = 256;              // blocks the stamp buffer has room for

enum OpKind { OP_QKV = 0, OP_O = 1, OP_GU = 2, OP_DOWN = 3, OP_HEAD = 4, N_OPS = 5 };

// One weight-streaming projection, cut into items = (k slice s, tile group g).
struct GemmOp {
    const bf16 *W1, *W2;     // layer-0 base; W2 only for the interleaved gate/up projection
    long long lstride;       // elements between layers
    int32_t N;               // weight rows in all (gate/up: 2F)
    int32_t MT;              // 16-row tiles
    int32_t K, S, KS;        // k extent, slices, slice length (multiple of 32)
    int32_t G, TPG;          // tile groups, tiles per group
    int32_t items, rot;      // S*G; block that gets item 0
    int32_t interleave;      // 1: tile t = gate rows 8t..8t+7 then up rows 8t..8t+7
};

struct Plan {
    GemmOp op[N_OPS];
    int32_t n_layers, has_head;
};

// Device buffers of the forward kernel beyond DevPtrs (all in the workspace).
struct FwdBufs {
    float *qkv;              // [MAX_ROWS][qrows] fp32, complete sums
    float *part;             // split-k partial tiles [S][MT][rpad][16]
    int32_t *tile_cnt;       // [MT max] arrivals per tile, zero between projections
    float *ssq;              // [d/16][MAX_ROWS] sum of squares of x over the 16 columns of a tile
    float *tile_top;         // [MT(head)][MAX_ROWS][4]: max, argmax (int bits), runner-up, unused
    float *attp;             // attention partials [item][MAX_ROWS][hd + 2]
    int32_t *att_cnt;        // [batch * H]
    unsigned long long *bar; // grid barrier counter
    int32_t *abort_flag;     // set when a bounded wait ran out
    unsigned long long *prof; // optional: every block stamps %globaltimer at its phase boundaries (NULL = off)
};

// ------------------------------------------------------------------ PTX helpers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *b, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *b, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *b, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    return ok != 0;
}
// global -> shared bulk copy; bytes a multiple of 16, both addresses 16-byte aligned
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long *p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ------------------------------------------------------------------ block-level context

struct Ctx {
    // shared memory
    unsigned char *scratch;        // SCRATCH_BYTES
    unsigned char *ring;           // this warp's stages
    uint64_t *mbar;                // this warp's STAGES barriers
    float *hand;                   // hand-over buffer of this warp pair
    uint64_t *hand_full, *hand_empty;
    int n_hand;                    // tiles handed over / received so far by this warp
    int32_t *row_pos, *row_tok;    // [MAX_ROWS]
    int32_t *n_rows;               // [MAX_ROWS] per sequence
    float *inv_rms;                // [MAX_ROWS]
    int32_t *flag;                 // block-wide scratch word
    // registers
    unsigned long long bar_target; // used by thread 0
    int warp, lane, cta, ncta;
    uint64_t policy;
};

// Grid barrier: every block arrives once; waits are bounded.  A wait that runs
// out raises the abort flag, after which all later barriers fall through.
__device__ __forceinline__ void grid_barrier(Ctx &c, const FwdBufs &fb) {
    __syncthreads();
    if (threadIdx.x == 0) {
        c.bar_target += (unsigned long long)c.ncta;
        __threadfence();
        atomicAdd(fb.bar, 1ULL);
        unsigned it = 0;
        while (ld_acquire_u64(fb.bar) < c.bar_target) {
            if (++it > SPIN_LIMIT || *(volatile int32_t *)fb.abort_flag) {
                atomicExch(fb.abort_flag, 1);
                break;
            }
        }
        __threadfence();
    }
    __syncthreads();
}

}  // namespace fwd
