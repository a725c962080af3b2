// One decoder forward as ONE persistent cooperative kernel (one block per SM).
//
// The forward is bound by streaming the weights from HBM once, so the kernel is
// built around an uninterrupted weight stream with as many bytes in flight as
// shared memory can hold, and a critical path with as few dependent
// global-memory round trips as possible:
//   - the weights are kept in HBM as 8-row x 64-column atoms (1 KB) that already
//     have the 128-byte-swizzled K-major layout tcgen05.mma reads from shared
//     memory, ordered [k block][row atom]: the rows a block owns in a projection
//     are one contiguous run per k block, fetched by ONE bulk async copy
//     (cp.async.bulk + mbarrier) into a byte ring; a producer thread walks the
//     static list of these stages for the WHOLE forward and runs ahead into the
//     next projection while the block sits in a grid barrier or a small phase;
//   - the contraction runs on the 5th-generation tensor cores: one thread issues
//     tcgen05.mma (M = 128, N = the block's weight rows, K = 16) with the
//     ACTIVATION rows as the A operand and the weight stage as the B operand, the
//     accumulator lives in tensor memory, and tcgen05.commit hands each stage back
//     to the producer the moment its MMAs are done, so nearly the whole ring is
//     in flight (a load takes about 3 us under full load: bandwidth = bytes in
//     flight / latency);
//   - activations enter as split bf16 (value rows, then remainder rows, stacked
//     along M), through a second small ring filled by activation-producer warps;
//   - the eight phase warps read the accumulator back (tcgen05.ld) into shared
//     memory once per projection and run the row-wise step that follows it in the
//     decoder (residual add, SwiGLU, bias/arg-max of the LM head) as the epilogue;
//     RMSNorm is split: the residual epilogue also writes x * gain as split bf16 in
//     operand order (the next projection's input) and the tile's share of
//     sum(x^2), and the 1/rms factor is applied to the OUTPUT rows of the next
//     projection in its epilogue, so no normalisation pass exists;
//   - phases are separated by grid barriers with bounded waits.
#pragma once
#include "common.cuh"

namespace fwd {

constexpr int MMA_WARPS = 8, MMA_THREADS = 256;  // warps 0..7 ("phase warps"): epilogues and all block-wide phases
constexpr int W_PRODUCER = 8, W_PRODUCERS = 3;   // lane 0 of warps 8, 10, 11: the weight stream, stage n by producer n % 3
constexpr int MMA_ISSUER = 9;                    // warp 9: owns the tensor memory; its lane 0 issues every tcgen05.mma
constexpr int X_PRODUCER = 12, X_PRODUCERS = 4;  // warps 12..14 provide the activation stages (stage s by producer s);
                                                 // warp 15 computes the RMS statistics
constexpr int THREADS = 32 * (X_PRODUCER + X_PRODUCERS);
constexpr int KB = 64;                          // k columns of a weight stage: one 128-byte swizzle row
constexpr int NB = 16;                          // weight stages that can be in flight (barrier pairs)
constexpr int RING_BYTES = 134 * 1024;          // weight ring of the forwards with at most 32 rows (a stage takes 128 B per
                                                // weight row of the block); wider forwards give part of it to the activations
constexpr int XS_MAX = 3;                       // activation stages: as many as fit, at most 3 (one producer warp each)
constexpr int XK = 256;                         // k columns of one activation stage (four k blocks)
// Per k block an activation stage holds NT atoms of bf16 values and then NT atoms of bf16 rounding remainders.
__host__ __device__ constexpr int xstage_bytes(int NT) { return (XK / KB) * 2 * NT * 1024; }
__host__ __device__ constexpr int x_stages(int NT) { return (80 * 1024) / xstage_bytes(NT) < XS_MAX ? (80 * 1024) / xstage_bytes(NT) : XS_MAX; }
constexpr int SCRATCH_BYTES = 88 * 1024;        // the activation ring lives in its first 72 KB at most; the epilogues' copy
                                                // of the accumulator, the attention phase and the tails use all of it
constexpr int MISC_BYTES = 5120;
constexpr int SMEM_BYTES = SCRATCH_BYTES + RING_BYTES + MISC_BYTES;    // the same total for every forward
static_assert(SMEM_BYTES <= 227 * 1024, "more shared memory than a block can have");   // (it is exactly that)
constexpr int MMA_TILES = 16;                   // 16-row tiles one tcgen05.mma covers (N = 256)
constexpr int MAX_TILES = 2 * MMA_TILES;        // tiles of one pass of a block: two accumulators, two MMAs per 16 k columns
                                                // (a block that has one tile too many for N = 256 still reads the activations once)
constexpr int ACC_COLS = 256;                   // fp32 accumulator columns of one accumulator (one per weight row)
constexpr int MAX_ROWS = 144;                   // rows of one forward (all sequences together): three groups of 48
constexpr int MAX_SEQ = 32;                     // sequences of one forward
constexpr int BIG_XBYTES = 144 * 1024;          // activation ring of a forward with more than 32 rows, at most
constexpr int MAX_SPLIT = 16;                   // key-range splits of one attention head
constexpr unsigned SPIN_LIMIT = 1u << 22;        // polls of a global word or a shared counter
constexpr unsigned MBAR_SPIN_LIMIT = 1u << 18;   // polls of an mbarrier (each may suspend for microseconds)
constexpr int PROF_STAMPS = 512;              // phase-boundary time stamps kept per block and forward
constexpr int PROF_BLOCKS = 256;              // blocks the stamp buffer has room for

enum OpKind { OP_QKV = 0, OP_O = 1, OP_GU = 2, OP_DOWN = 3, OP_HEAD = 4, N_OPS = 5 };

// One weight-streaming projection.  Block c owns the contiguous tiles
// [t0, t0 + T) given by op_range(); it runs them in passes of at most MAX_TILES, evenly sized.
struct GemmOp {
    const bf16 *W;           // layer-0 base of the tiled weights: [K/64][2*MT atoms][8 rows][64 k, 16-byte chunks XOR-swizzled by row]
    const bf16 *X;           // activations, split bf16 in operand order (see xatom_index)
    long long lstride;       // elements between layers
    int32_t N;               // weight rows in all (gate/up: 2F)
    int32_t MT;              // 16-row tiles
    int32_t K;
    int32_t S;               // k slices: 1, or (attention output / MLP down, which have few tiles) a divisor of the
                             // grid size: the slices' partial tiles are summed by a small pass after a grid barrier
    int32_t rot;             // block that gets the first tile range (spreads the one-tile imbalance)
};

struct Plan {
    GemmOp op[N_OPS];
    int32_t n_layers, has_head;
    int32_t max_tiles;       // tiles of one pass: MMA_TILES, or MAX_TILES in the kernel variant with two accumulators
                             // (10 with three row groups: their accumulators share the 512 tensor-memory columns)
    // shared-memory plan (bytes): [activation ring / scratch][weight ring][barriers and row tables]
    int32_t scratch_bytes, ring_bytes;
    int32_t xkb;             // 64-column k blocks per activation stage
    int32_t xs;              // activation stages
    int32_t xkb_bytes;       // bytes of one k block of activations: 2 KB per eight-row tile (values + remainders)
    int32_t acc_stride;      // tensor-memory columns between the accumulators of two row groups
};

// Device buffers of the forward kernel beyond DevPtrs (all in the workspace).
struct FwdBufs {
    float *qkv;              // [k slices][MAX_ROWS][qrows] fp32
    bf16 *xg;                // x * gain of the next RMSNorm, split bf16 in operand order (its 1/rms comes later)
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

// ---- 5th-generation tensor cores (tcgen05) and tensor memory

// Shared-memory matrix descriptor of a K-major operand in the 128-byte swizzle layout: rows of 128 bytes, groups of
// eight rows 1024 bytes apart; `saddr` is 1024-byte aligned plus 32 bytes per 16-column step inside the swizzle row.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n (a multiple of 16, at most 256).
__device__ __forceinline__ uint32_t umma_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)n >> 3) << 17) | ((128u >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]^T, issued by one thread.
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
                 ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
// The barrier gets one arrival when every tcgen05.mma this thread issued before has finished.
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 32 consecutive accumulator columns of this thread's lane (lane = 32 * (warp % 4) + lane id).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
                   "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]),
                   "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
                   "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ------------------------------------------------------------------ block-level context

struct Ctx {
    // shared memory
    unsigned char *scratch;        // SCRATCH_BYTES (activation ring in front)
    unsigned char *ring;           // weight ring
    int ring_bytes;
    uint64_t *wfull, *wempty;      // [NB]
    uint64_t *xfull, *xempty;      // [XS_MAX]
    uint64_t *acc_full, *acc_empty; // the accumulator of a pass is complete / has been copied out
    volatile int32_t *pass_done;   // passes whose epilogue is over (the activation ring may be overwritten)
    uint32_t tmem;                 // tensor-memory address of the accumulator
    int32_t *row_pos, *row_tok;    // [MAX_ROWS]
    int32_t *n_rows;               // [MAX_SEQ] per sequence
    int32_t *key_start;            // [MAX_SEQ] per sequence: first cache position the rows attend to (0 unless the
                                   // pre-verification model runs with a restricted attention context)
    float *inv_rms;                // [MAX_ROWS]
    volatile int32_t *ready_op;    // [0] projections whose inputs are complete; [1] projections whose inv_rms is ready
    int32_t *flag;                 // block-wide scratch word
    // registers
    unsigned long long bar_target; // used by thread 0
    int warp, lane, cta, ncta;
    uint64_t policy;
    int np;                        // passes of this block finished so far (phase warps)
};

// Activations enter the tensor cores as TWO bf16 numbers, hi = bf16(v) and lo = bf16(v - hi): together they carry
// 16 mantissa bits, so rounding the inputs of a projection no longer shows in the logits (with single bf16 inputs
// the error against an fp64 evaluation grows to 0.18 over 32 layers of width 4096).  The weights stay bf16 as given.
//
// Operand order of an activation buffer with nt row tiles of 8: [k / 64][2 * nt atoms][8 rows][64 k], an atom being
// 1 KB in the 128-byte swizzle layout (the 16-byte chunk c of row r sits at chunk c ^ r); atoms 0 .. nt-1 of a
// k block hold the values of rows 8a .. 8a+7, atoms nt .. 2nt-1 the remainders.  As the A operand of an MMA with
// M = 128 the values are accumulator lanes 0 .. 8nt-1 and the remainders lanes 8nt .. 16nt-1; the epilogue adds them.
//
// With more than 64 rows the rows form G groups of 8 * nt rows; a k block then holds the groups one after the other
// (each its values, then its remainders), and every group is the A operand of its own MMA and accumulator.
struct XLay {
    int nt, G;                     // eight-row tiles per group, groups
};
__device__ __forceinline__ size_t xatom_index(int r, int k, XLay x, int plane) {
    const int kk = k & 63, rr = r & 7, rg = 8 * x.nt, g = x.G == 1 ? 0 : r / rg, rl = r - g * rg;   // (one group: no division)
    return ((size_t)(k >> 6) * (2 * x.nt * x.G) + g * (2 * x.nt) + plane * x.nt + (rl >> 3)) * 512 + rr * 64 +
           ((((kk >> 3) ^ rr) << 3) | (kk & 7));
}
__device__ __forceinline__ void store_split(bf16 *base, XLay x, int r, int k, float v) {
    const bf16 h = __float2bfloat16(v);
    base[xatom_index(r, k, x, 0)] = h;
    base[xatom_index(r, k, x, 1)] = __float2bfloat16(v - __bfloat162float(h));
}

// Barrier of the eight phase warps (the producer warps never join it).
__device__ __forceinline__ void bsync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Work of block `cta` in a projection: tiles [t0, t0 + T) over the k range [k_lo, k_hi).
// With S slices the blocks form ncta / S groups; a group shares a tile range and its S
// blocks take one k slice each (slices are whole 64-column k blocks, as even as they come).
__device__ __host__ __forceinline__ void op_range(const GemmOp &op, int cta, int ncta, int &t0, int &T, int &k_lo, int &k_hi) {
    int ci = cta - op.rot;
    if (ci < 0) ci += ncta;
    const int groups = ncta / op.S, g = ci / op.S, s = ci % op.S;
    const int base = op.MT / groups, rem = op.MT % groups;
    T = g < groups ? base + (g < rem ? 1 : 0) : 0;
    t0 = g * base + (g < rem ? g : rem);
    const int nks = op.K / KB, sb = nks / op.S, sr = nks % op.S;
    k_lo = (s * sb + (s < sr ? s : sr)) * KB;
    k_hi = k_lo + (sb + (s < sr ? 1 : 0)) * KB;
    if (k_hi > op.K) k_hi = op.K;
    if (k_lo >= k_hi) T = 0;
}

// Passes of a block over its T tiles: as few as possible, evenly sized (the activations are streamed
// once per pass, and an even split keeps every pass bandwidth bound rather than latency bound).
__device__ __host__ __forceinline__ int n_passes(int T, int cap) { return (T + cap - 1) / cap; }
__device__ __host__ __forceinline__ void pass_range(int T, int p, int cap, int &p0, int &Tp) {
    const int np = n_passes(T, cap), base = T / np, rem = T % np;
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
