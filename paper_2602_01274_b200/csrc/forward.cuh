// One decoder forward as ONE persistent cooperative kernel (one block per SM).
//
// The forward is bound by streaming the weights from HBM once, so the kernel is
// built around an uninterrupted weight stream and a critical path with as few
// dependent global-memory round trips as possible:
//   - a producer warp walks the static list of weight units (16 rows x 256 k)
//     of the block for the WHOLE forward and keeps a shared-memory ring full
//     with bulk async copies (cp.async.bulk + mbarrier); it runs ahead into the
//     next projection while the block sits in a grid barrier or in a small
//     phase, so the HBM queue never drains between projections;
//   - a block owns whole 16-row tiles of a projection over its k range (no
//     partial-sum buffers, no arrival counters, no fences), the eight MMA warps
//     advance over k in lockstep, and the activation rows of each 256-wide k
//     step arrive through a second small ring, filled by activation-producer warps;
//   - tensor cores (mma.m16n8k16, bf16 in / fp32 accumulate, weights as the
//     16-row operand) do the contraction, so the math is invisible;
//   - the row-wise step that follows a projection in the decoder (residual add,
//     SwiGLU, bias/arg-max of the LM head) is the epilogue of the warp that owns
//     the tile; RMSNorm is split: the residual epilogue also writes x * gain as
//     bf16 in fragment order (the next projection's input) and the tile's share
//     of sum(x^2), and the 1/rms factor is applied to the OUTPUT rows of the
//     next projection in its epilogue, so no normalisation pass exists;
//   - phases are separated by grid barriers with bounded waits.
#pragma once
#include "common.cuh"

namespace fwd {

constexpr int MMA_WARPS = 8, MMA_THREADS = 256;  // warps 0..7: MMAs, epilogues and all block-wide phases
constexpr int W_PRODUCERS = 4;                   // warps 8..11 stream weights: unit n by producer n % 4 (one warp alone
                                                 // cannot issue the bulk copies fast enough)
constexpr int X_PRODUCERS = 4;                   // warps 12..14 provide the activation chunks (stage s by producer s); warp 15
                                                 // computes the RMS statistics
constexpr int W_PRODUCER = MMA_WARPS, X_PRODUCER = W_PRODUCER + W_PRODUCERS;
constexpr int THREADS = 32 * (X_PRODUCER + X_PRODUCERS);
constexpr int KC = 512;                         // k columns of one weight unit: 1 KB per row and copy (DRAM likes long runs)
constexpr int PITCH = KC * 2 + 64;              // bytes between the rows of a stage (bank-conflict free)
constexpr int STAGE_BYTES = 16 * PITCH;         // 17408
constexpr int NS = 8;                           // weight stages in the ring: one wave of the eight MMA warps
constexpr int RING_BYTES = NS * STAGE_BYTES;    // 139264
constexpr int XS_MAX = 3;                       // activation stages: as many as fit the scratch, at most 3 (one producer warp each)
constexpr int XK = 256;                         // k columns of one activation chunk (half a weight unit)
constexpr int XCH = XK / 32;                    // its 32-wide chunks
// An activation stage holds one chunk twice: the bf16 value ("hi") and the bf16 rounding remainder ("lo").
__host__ __device__ constexpr int xstage_bytes(int NT) { return 2 * NT * XCH * 512; }   // hi + lo, row tiles x chunks x 512 B
__host__ __device__ constexpr int x_stages(int NT) { return (80 * 1024) / xstage_bytes(NT) < XS_MAX ? (80 * 1024) / xstage_bytes(NT) : XS_MAX; }
constexpr int SCRATCH_BYTES = 88 * 1024;        // the activation ring lives in its first 48 KB; the attention
                                                // phase and the tails use all of it (no activations in flight then)
constexpr int MISC_BYTES = 2048;
constexpr int SMEM_BYTES = SCRATCH_BYTES + RING_BYTES + MISC_BYTES;
constexpr int MAX_TILES = 8;                    // tiles of one pass of a block: one per MMA warp, one ring generation per k step
constexpr int MAX_ROWS = 32;                    // rows of one forward (all sequences together)
constexpr int MAX_SPLIT = 16;                   // key-range splits of one attention head
constexpr unsigned SPIN_LIMIT = 1u << 22;        // polls of a global word or a shared counter
constexpr unsigned MBAR_SPIN_LIMIT = 1u << 18;   // polls of an mbarrier (each may suspend for microseconds)
constexpr int PROF_STAMPS = 512;              // phase-boundary time stamps kept per block and forward
constexpr int PROF_BLOCKS = 256;              // blocks the stamp buffer has room for

enum OpKind { OP_QKV = 0, OP_O = 1, OP_GU = 2, OP_DOWN = 3, OP_HEAD = 4, N_OPS = 5 };

// One weight-streaming projection.  Block c owns the contiguous tiles
// [t0, t0 + T) given by op_range(); it runs them in passes of at most MAX_TILES, evenly sized.
struct GemmOp {
    const bf16 *W1, *W2;     // layer-0 base; W2 only for the interleaved gate/up projection
    const bf16 *X;           // activations, bf16 in fragment order [K/32][row tiles][32 lanes][8]: the values rounded to bf16
    long long x_lo;          // element offset from X to the same layout holding the rounding remainders (also bf16)
    long long lstride;       // elements between layers
    int32_t N;               // weight rows in all (gate/up: 2F)
    int32_t MT;              // 16-row tiles
    int32_t K;
    int32_t S;               // k slices: 1, or (attention output / MLP down, which have few tiles) a divisor of the
                             // grid size: the slices' partial tiles are summed by a small pass after a grid barrier
    int32_t rot;             // block that gets the first tile range (spreads the one-tile imbalance)
    int32_t interleave;      // 1: tile t = gate rows 8t..8t+7 then up rows 8t..8t+7
};

struct Plan {
    GemmOp op[N_OPS];
    int32_t n_layers, has_head;
};

// Device buffers of the forward kernel beyond DevPtrs (all in the workspace).
struct FwdBufs {
    float *qkv;              // [MAX_ROWS][qrows] fp32
    bf16 *xg;                // x * gain of the next RMSNorm, split bf16 in fragment order (its 1/rms comes later)
    long long xg_lo, att_lo, act_lo;   // element offsets of the remainder halves of xg, DevPtrs::att, DevPtrs::act
    float *ssq;              // [d/16][MAX_ROWS] sum of squares of x over the 16 columns of a tile
    float *part;             // k-slice partial tiles [S][d/16][row tiles * 8][16] of the two residual projections
    float *tile_top;         // [MT(head)][MAX_ROWS][4]: max, argmax (int bits), runner-up, unused
    float *attp;             // attention partials [seq*H + h][split][row][hd + 2]
    int32_t *att_cnt;        // [batch * H]
    unsigned long long *bar; // grid barrier counter
    int32_t *abort_flag;     // [0] code of the first bounded wait that ran out, [1..3] its block, warp, detail
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
    unsigned char *scratch;        // SCRATCH_BYTES (activation ring in front)
    unsigned char *ring;           // weight ring
    uint64_t *wfull, *wempty;      // [NS]
    uint64_t *xfull, *xempty;      // [XS_MAX]
    int32_t *row_pos, *row_tok;    // [MAX_ROWS]
    int32_t *n_rows;               // [MAX_ROWS] per sequence
    float *inv_rms;                // [MAX_ROWS]
    volatile int32_t *ready_op;    // [0] projections whose inputs are complete; [1] projections whose inv_rms is ready
    int32_t *flag;                 // block-wide scratch word
    // registers
    unsigned long long bar_target; // used by thread 0
    int warp, lane, cta, ncta;
    uint64_t policy;
    int wn, xn;                    // weight units / activation chunks of this block consumed (or produced) so far
};

// Activations enter the tensor cores as TWO bf16 numbers, hi = bf16(v) and lo = bf16(v - hi): together they carry
// 16 mantissa bits, so rounding the inputs of a projection no longer shows in the logits (with single bf16 inputs
// the error against an fp64 evaluation grows to 0.18 over 32 layers of width 4096).  The weights stay bf16 as given.
__device__ __forceinline__ void store_split(bf16 *hi_base, long long lo_off, size_t idx, float v) {
    const bf16 h = __float2bfloat16(v);
    hi_base[idx] = h;
    hi_base[idx + lo_off] = __float2bfloat16(v - __bfloat162float(h));
}

// Barrier of the eight MMA warps (the producer warps never join it).
__device__ __forceinline__ void bsync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Work of block `cta` in a projection: tiles [t0, t0 + T) over the k range [k_lo, k_hi).
// With S slices the blocks form ncta / S groups; a group shares a tile range and its S
// blocks take one k slice each (slices are whole KC steps).
__device__ __host__ __forceinline__ void op_range(const GemmOp &op, int cta, int ncta, int &t0, int &T, int &k_lo, int &k_hi) {
    int ci = cta - op.rot;
    if (ci < 0) ci += ncta;
    const int groups = ncta / op.S, g = ci / op.S, s = ci % op.S;
    const int base = op.MT / groups, rem = op.MT % groups;
    T = g < groups ? base + (g < rem ? 1 : 0) : 0;
    t0 = g * base + (g < rem ? g : rem);
    const int nks = (op.K + KC - 1) / KC, sb = nks / op.S, sr = nks % op.S;
    k_lo = (s * sb + (s < sr ? s : sr)) * KC;
    k_hi = k_lo + (sb + (s < sr ? 1 : 0)) * KC;
    if (k_hi > op.K) k_hi = op.K;
    if (k_lo >= k_hi) T = 0;
}

// Passes of a block over its T tiles: as few as possible, evenly sized (the activations are streamed
// once per pass, and an even split keeps every pass bandwidth bound rather than latency bound).
__device__ __host__ __forceinline__ int n_passes(int T) { return (T + MAX_TILES - 1) / MAX_TILES; }
__device__ __host__ __forceinline__ void pass_range(int T, int p, int &p0, int &Tp) {
    const int np = n_passes(T), base = T / np, rem = T % np;
    Tp = base + (p < rem ? 1 : 0);
    p0 = p * base + (p < rem ? p : rem);
}

// k slice of block `cta` in a sliced projection.
__device__ __host__ __forceinline__ int op_slice(const GemmOp &op, int cta, int ncta) {
    int ci = cta - op.rot;
    if (ci < 0) ci += ncta;
    return ci % op.S;
}

// Grid barrier (MMA warps only): every block arrives once; waits are bounded.  A wait that runs
// out raises the abort flag, after which all later barriers fall through.
__device__ __forceinline__ void grid_barrier(Ctx &c, const FwdBufs &fb) {
    asm volatile("fence.proxy.async;" ::: "memory");   // this thread's global writes, for bulk copies issued later
    bsync();
    if (threadIdx.x == 0) {
        c.bar_target += (unsigned long long)c.ncta;
        __threadfence();
        atomicAdd(fb.bar, 1ULL);
        unsigned it = 0;
        while (ld_acquire_u64(fb.bar) < c.bar_target) {
            ++it;
            if ((it & 255u) == 0 && (it > 4u * SPIN_LIMIT || *(volatile int32_t *)fb.abort_flag)) {
                atomicCAS(fb.abort_flag, 0, 1);
                break;
            }
        }
        __threadfence();
    }
    bsync();
}

}  // namespace fwd
