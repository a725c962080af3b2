/*
 * pacer.h - C ABI of the B200 (sm_100a) hot path of Pacer: speculative decoding
 * in which a draft model decodes in blocks of b tokens, a one-layer
 * pre-verification model scores every block and stops the drafting when a block
 * fails, the target model verifies all drafts in one forward over its KV cache,
 * and an acceptance step commits a prefix of the drafts and rolls the caches back.
 *
 * Conventions
 *   - Every function returns 0 (PACER_OK) or a negative PACER_E* code; nothing
 *     throws, aborts or traps the device.  pacer_strerror(code) and
 *     pacer_last_error(ctx) give text.
 *   - "device" pointers are CUDA device addresses on the current device, "host"
 *     pointers are ordinary memory.  All device memory is CALLER-OWNED: the
 *     library never allocates or frees device memory.  It carves the workspace
 *     given to pacer_create; pacer_load_weights copies the projection matrices
 *     into it in the order the forward kernel streams them (the workspace holds
 *     one copy of every layer matrix and LM head) and reads the other tensors in
 *     place.
 *   - Calls enqueue work on the context's stream and return without waiting
 *     unless marked [sync].  A context is not thread-safe.
 *   - Models are Llama-style decoders: RMSNorm, rotary embedding (rotate-half,
 *     absolute positions), causal attention with n_kv_heads <= n_heads, SwiGLU
 *     MLP, untied embedding and LM head, no biases.  Weights are bf16, matrices
 *     are [out][in] row-major and stacked over layers; accumulation, the residual
 *     stream, norms and softmax are fp32.  Activations enter the tensor cores as
 *     a bf16 value plus a bf16 rounding remainder (16 mantissa bits), and the KV
 *     caches hold both parts.
 *   - Batch rows are independent sequences.  Token ids are int32.
 */
#ifndef PACER_H_
#define PACER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    PACER_OK = 0,
    PACER_EINVAL = -1,       /* bad argument (null pointer, size out of range, shape mismatch) */
    PACER_ENOMEM = -2,       /* workspace too small */
    PACER_ECUDA = -3,        /* a CUDA runtime call failed; see pacer_last_error */
    PACER_EDEVICE = -4,      /* a kernel reported an anomaly in the device status word */
    PACER_ESTATE = -5,       /* call out of order (weights missing, no prefill, ...) */
    PACER_EUNSUPPORTED = -6
};

typedef struct pacer_ctx pacer_ctx;

/* d_model and d_ffn are multiples of 64 (the width of a weight stage), d_model / n_heads is 64 or 128. */
typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, d_ffn, vocab;
    float rope_theta;        /* 10000 */
    float rms_eps;           /* 1e-5 */
} pacer_model_cfg;

typedef struct {
    pacer_model_cfg target, draft;   /* the pre-verification model M_B is ONE layer with the draft's widths */
    int32_t max_batch;       /* sequences decoded together */
    int32_t max_ctx;         /* cache rows per sequence: n_prompt + max_new + gamma_cap + 2 must fit */
    int32_t gamma_cap;       /* largest draft window; a multiple of block_b */
    int32_t block_b;         /* drafts per pre-verification block (paper: b) */
    float rho;               /* threshold growth per passed block (paper: rho > 1) */
    int32_t criterion;       /* block statistic: 0 mean (the method), 1 minimum ("any"), 2 last token */
    float succ_bias;         /* added to logit succ[input token] of every LM-head row; 0 = off */
    int32_t use_posemb;      /* 1: add the draft position embedding e_i (the method); 0: ablation */
    int32_t mb_scope;        /* attention context of M_B ("attention context" ablation): 0 full = its whole KV cache
                                (the method), 1 local draft = the drafts of the current step, 2 local block = the
                                drafts of the current block.  A restricted context starts at the first draft row of
                                the step / block; history rows are outside it and attend to themselves only. */
} pacer_cfg;

/* One named weight tensor, bf16, contiguous, on the device.  Names per model:
 *   embed [V][d]            wqkv [L][(H+2Hkv)*hd][d]  (q rows, then k, then v)
 *   wo [L][d][H*hd]         wgate, wup [L][F][d]       wdown [L][d][F]
 *   norm1, norm2 [L][d]     normf [d]                  head [V][d]
 * M_B (which = 2) has no embed/head but  head_b [2][d]  and  posemb [gamma_cap][d].
 * wqkv, wo, wgate, wup, wdown and head are copied (re-laid for the tensor cores) by
 * pacer_load_weights and may be freed once the stream has run it; embed, the norm
 * gains, head_b and posemb are used in place and must outlive the context. */
typedef struct {
    const char *name;
    const void *dev_ptr;
    int64_t numel;
} pacer_tensor;

enum { PACER_TARGET = 0, PACER_DRAFT = 1, PACER_PREVERIFY = 2 };
enum { PACER_GREEDY = 0, PACER_SAMPLE = 1 };

/* Counters and device-side timings of one pacer_generate / pacer_generate_ar call. */
typedef struct {
    int64_t n_draft_fwd, n_mb_calls, n_target_fwd, n_steps;  /* summed over sequences */
    int64_t n_generated;        /* tokens committed, summed over sequences (before truncation to max_new) */
    int64_t n_kernel_launches;  /* kernels of this library launched inside the timed decode region */
    float ms_prefill;           /* CUDA-event time of the prefill */
    float ms_decode;            /* CUDA-event time of the decode loop (first step .. last step) */
} pacer_stats;

/* Per-sequence scalars copied out by pacer_read_state. */
typedef struct {
    int32_t P;                  /* accepted tokens so far, prompt included */
    int32_t len_T, len_D, len_B;/* rows in the target / draft / M_B caches */
    int32_t gamma;              /* drafts made in the current step */
    int32_t k_round;            /* blocks that passed pre-verification in the current step */
    float t_k;                  /* current threshold t_0 * rho^k */
    int32_t drafting;           /* 1 while the draft loop of this step may continue */
    int32_t finished;           /* 1 once max_new tokens exist */
    int32_t n_steps;            /* draft-and-verify steps completed */
    int32_t last_n, last_next;  /* accepted drafts and the follow-up token of the last step */
    int32_t n_pend;             /* draft hidden rows not yet given to M_B */
    int32_t err;                /* unused, 0 (the device status word is per context: PACER_EDEVICE) */
    int64_t n_draft_fwd, n_mb_calls, n_target_fwd;
} pacer_seq_state;

/* Device buffers that pacer_read_buffer can copy out (stage-by-stage checks). */
enum {
    PACER_BUF_TOKENS = 0,        /* int32 [max_batch][max_ctx]   accepted tokens x */
    PACER_BUF_DRAFTS = 1,        /* int32 [max_batch][gamma_cap] y_1..y_gamma of the current step */
    PACER_BUF_ALPHA = 2,         /* f32   [max_batch][gamma_cap] alpha_hat of the current step's drafts */
    PACER_BUF_VERIFY_LOGITS = 3, /* f32   [max_batch][gamma_cap+1][V] target logits of the last verify */
    PACER_BUF_DRAFT_LOGITS = 4,  /* f32   [max_batch][gamma_cap][V] draft logits q_i of the current step */
    PACER_BUF_HPEND = 5,         /* f32   [max_batch][block_b+1][d_draft] hidden rows waiting for M_B */
    PACER_BUF_DRAFT_LEN = 6,     /* int32 [max_batch][max_steps] gamma of every step */
    PACER_BUF_ACCEPT_LEN = 7,    /* int32 [max_batch][max_steps] n of every step */
    PACER_BUF_KCACHE_T = 8,      /* bf16  [2][L][max_batch][Hkv][max_ctx][hd]: the values rounded to bf16, then their rounding
                                    remainders (value - bf16(value), also bf16)  (also _D = 10, _B = 12) */
    PACER_BUF_VCACHE_T = 9,      /* bf16  same shape                        (also _D = 11, _B = 13) */
    PACER_BUF_KCACHE_D = 10, PACER_BUF_VCACHE_D = 11, PACER_BUF_KCACHE_B = 12, PACER_BUF_VCACHE_B = 13,
    PACER_BUF_PHASE_NS = 14      /* u64 [256 blocks][512] device clock (ns) at the phase boundaries of the last
                                    forward run while profiling (any model), per block: start, input rows, barrier, then per
                                    layer QKV, barrier, attention, barrier, O, barrier, gate/up, barrier, down,
                                    barrier; LM head, barrier; end (at most 512 stamps are kept) */
};

const char *pacer_strerror(int code);
const char *pacer_last_error(const pacer_ctx *ctx);

/* Bytes of device workspace a context with this configuration needs (the
 * re-laid projection matrices and KV caches of the three models, activations,
 * logits, per-sequence state).  0 on a bad configuration. */
size_t pacer_workspace_bytes(const pacer_cfg *cfg);

/* Creates a context on the current device.  dev_workspace: device, at least
 * pacer_workspace_bytes(cfg) bytes, 256-byte aligned, caller-owned, must outlive
 * the context.  cuda_stream: a cudaStream_t (NULL = the legacy default stream).
 * Allocates host memory only.  Zeroes the state part of the workspace. */
int pacer_create(const pacer_cfg *cfg, void *dev_workspace, size_t workspace_bytes, void *cuda_stream,
                 pacer_ctx **out);

/* Frees host memory and CUDA events/graphs of the context; the workspace and the
 * weights stay untouched.  [sync] */
int pacer_destroy(pacer_ctx *ctx);

/* Registers the weights of one model (which = PACER_TARGET / _DRAFT / _PREVERIFY).
 * tbl: host array of n entries naming device tensors (see pacer_tensor); numel is
 * checked against the configuration.  succ: device int32 [V] planted successor
 * table for the LM-head bias, or NULL (ignored for M_B). */
int pacer_load_weights(pacer_ctx *ctx, int which, const pacer_tensor *tbl, int n, const int32_t *succ);

/* Starts `batch` sequences from prompts (host int32 [batch][n_prompt]) and fills
 * the three caches with prompt tokens 0..n_prompt-2; the last prompt token is the
 * first step's input row (the prefix x of Algorithm 1).  The hidden states the
 * draft produces for the prompt are M_B's history h_x (Eq. 7), without position
 * embedding.  threshold / mode / seed / max_new configure the steps that follow:
 * threshold < 0 means the block test always passes (fixed window gamma_max).
 * gamma_max is rounded down to a multiple of block_b and must be in
 * [block_b, gamma_cap]. */
int pacer_prefill(pacer_ctx *ctx, const int32_t *prompt, int batch, int n_prompt, int max_new, int gamma_max,
                  float threshold, int mode, uint64_t seed);

/* One draft-model forward for every sequence that is still drafting (Eq. 6, one
 * of the b steps of a block): emits y_i (argmax, or a Gumbel-max draw when
 * sampling), keeps the logits q_i and queues the hidden state h_i for M_B.  The
 * first forward after a fully accepted step takes two rows (the draft cache
 * lacks the last draft of that step). */
int pacer_draft_step(pacer_ctx *ctx);

/* Pre-verification of the rows queued since the last call (Eq. 7): M_B on
 * [h_i + e_i] against its own KV cache gives alpha_hat_i; then the block test of
 * Algorithm 1: drafting stops when the block statistic <= t_k or the window is
 * full, else t_{k+1} = t_k * rho. */
int pacer_preverify(pacer_ctx *ctx);

/* One target forward over [last accepted token, y_1..y_gamma] per sequence
 * (Eq. 4), appending their K/V rows and leaving logits p_1..p_{gamma+1}. */
int pacer_verify(pacer_ctx *ctx);

/* Acceptance after a pacer_verify call (Eq. 5; greedy = prefix match with the target's argmax), commit of
 * [y_1..y_n, next], truncation of the three caches to the accepted rows, reset of
 * the per-step state, logging of (gamma, n). Uses the mode and seed of pacer_prefill. */
int pacer_accept_rollback(pacer_ctx *ctx);

/* Test hook for the error path: writes the device status word exactly as a kernel's
 * bounded wait that ran out would (code != 0, and the block, warp and detail it
 * records).  Until the next pacer_prefill / pacer_generate* resets the word, every
 * [sync] entry point returns PACER_EDEVICE with the decoded text, and forwards
 * launched meanwhile fall through their waits.  No kernel is launched.  [sync] */
int pacer_debug_set_device_status(pacer_ctx *ctx, int code, int block, int warp, int detail);

/* [sync] Copies the per-sequence scalars of sequences 0..batch-1 to host memory.
 * Returns PACER_EDEVICE (after filling `out`) when the device status word is set. */
int pacer_read_state(pacer_ctx *ctx, pacer_seq_state *out, int batch);

/* [sync] Copies `bytes` bytes from the start of one device buffer (PACER_BUF_*) to host memory.
 * Returns PACER_EDEVICE (after the copy) when the device status word is set. */
int pacer_read_buffer(pacer_ctx *ctx, int which, void *host_dst, size_t bytes);

/* [sync] Algorithm 1 end to end: prefill, then draft-and-verify steps until every
 * sequence has max_new new tokens.  Every decision of the loop (rows of a forward,
 * stop of the drafting, acceptance, rollback, end of generation) is taken on the
 * device; the host enqueues whole steps (every block of the window, each a no-op
 * for a sequence that has stopped drafting) and stays two steps ahead of the device:
 * it reads the finished flags of an EARLIER step from pinned memory (copied there
 * behind an event) to know when to stop enqueuing, and never waits for the step it
 * has just enqueued.  The launches of one step (the draft forwards and pre-verification
 * calls of the whole window, the verify forward, the acceptance) are captured once
 * per context as a CUDA graph and replayed every step (not on the legacy default
 * stream, which cannot be captured: there the launches are issued one by one).  Greedy runs take the
 * acceptance (Eq. 5) in the tail of the verify forward; sampling runs in a kernel of
 * its own.
 * Outputs, all host, caller-owned:
 *   out_tokens     int32 [batch][max_new]
 *   out_n_steps    int32 [batch]
 *   out_draft_len  int32 [batch][max_new]  gamma of step s, -1 beyond n_steps
 *   out_accept_len int32 [batch][max_new]  n of step s, -1 beyond n_steps
 *   stats          may be NULL */
int pacer_generate(pacer_ctx *ctx, const int32_t *prompt, int batch, int n_prompt, int max_new, int gamma_max,
                   float threshold, int mode, uint64_t seed, int32_t *out_tokens, int32_t *out_n_steps,
                   int32_t *out_draft_len, int32_t *out_accept_len, pacer_stats *stats);

/* [sync] Speculative decoding (Section 2.2) with the draft window of every step
 * PRESCRIBED instead of decided by the pre-verification model: step s of sequence q
 * drafts windows[q][s] tokens (host int32 [batch][n_windows], each in [0, gamma_cap];
 * 0 = a plain target step; steps beyond n_windows reuse the last entry).  With
 * windows = the accepted lengths of a large-window run of the same prompt this is
 * decoding with the optimal draft length gamma* of Section 3.1 (the upper bound an
 * oracle-knowledge window reaches).  M_B is not run.  The draft model catches up, in
 * the first forward of its next window, on the rows it has not seen; such a forward
 * holds at most 16 rows per sequence (32 / batch if that is less), and when the
 * backlog reaches that number a prescribed 0 becomes 1.  Outputs as pacer_generate. */
int pacer_generate_sched(pacer_ctx *ctx, const int32_t *prompt, int batch, int n_prompt, int max_new,
                         const int32_t *windows, int n_windows, int mode, uint64_t seed, int32_t *out_tokens,
                         int32_t *out_n_steps, int32_t *out_draft_len, int32_t *out_accept_len, pacer_stats *stats);

/* [sync] Autoregressive decoding of the target alone on the same kernels (Eq. 1):
 * the baseline, and under greedy decoding the definition of the lossless output. */
int pacer_generate_ar(pacer_ctx *ctx, const int32_t *prompt, int batch, int n_prompt, int max_new, int mode,
                      uint64_t seed, int32_t *out_tokens, pacer_stats *stats);

/* Kernel-level timing for roofline reports.  Between pacer_profile_begin and
 * pacer_profile_end every forward of the TARGET model (one launch of the
 * persistent forward kernel) is bracketed by a pair of CUDA events on the
 * context's stream (at most 4096 launches are recorded; later ones run untimed)
 * and every block of every forward (any model) stamps the device clock at its phase
 * boundaries (PACER_BUF_PHASE_NS keeps the last forward's).  pacer_profile_end [sync] returns the summed device time
 * of those launches (ms), the bf16 weight bytes they streamed and their count.
 * Whole-loop timings are taken without it. */
int pacer_profile_begin(pacer_ctx *ctx);
int pacer_profile_end(pacer_ctx *ctx, double *fwd_ms, double *fwd_weight_bytes, int64_t *fwd_launches);

/* Y[r][n] = sum_k X[r][k] * W[n][k]: a stand-alone skinny weight-streaming product
 * (a split-k kernel on mma.sync with plain bf16 activations; the projections inside
 * the forwards run on a different, tcgen05 path with split activations).  x: device bf16
 * [rows][K] row-major; w: device bf16 [N][K]; y: device f32 [rows][N];
 * scratch: device, at least pacer_linear_scratch_bytes(rows, N, K) bytes.
 * rows <= 32, K a multiple of 32.  Enqueues on `cuda_stream`. */
size_t pacer_linear_scratch_bytes(int rows, int N, int K);
int pacer_linear(const void *x, const void *w, float *y, int rows, int N, int K, void *scratch,
                 size_t scratch_bytes, void *cuda_stream);

/* The same product as pacer_linear for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a service entry point of the library.)
 * Who needs it: a serving process that handed all device memory to its own arena
 * at start-up, or a plug-in host without an allocator of its own, has nothing to
 * offer as `scratch`, and a cudaMalloc inside the decode loop would stall the whole
 * device (it synchronises) or simply fail once the arena owns the memory.  Here the
 * scratch is a fixed array of PACER_LINEAR_STATIC_BYTES bytes inside the library
 * image; every GPU that loads the library holds it until the process exits.
 *   - x, w, y, rows, N, K, cuda_stream: exactly as pacer_linear; inputs and the
 *     output remain caller-owned device memory.
 *   - Shapes whose pacer_linear_scratch_bytes(rows, N, K) exceeds
 *     PACER_LINEAR_STATIC_BYTES are refused with PACER_ENOMEM before any launch.
 *   - No cudaMalloc, cudaFree or allocating library routine is called, ever.
 *   - The first call on each device looks up the device address of the array
 *     (cudaGetSymbolAddress, with that device current) and remembers it; make that
 *     first call before starting any stream capture on the device.
 *   - All calls on one device share the one array, which keeps whatever the last
 *     call left in it.  Nothing in it has to start at zero: the kernels overwrite
 *     every element they later read.  Two calls that overlap on the GPU (different
 *     streams, no ordering between them) race on the array; order them.
 *   - Host threads: the per-device address table is filled without a lock, so the first
 *     calls on a device must not come from two host threads at once; later calls only
 *     read it. */
#define PACER_LINEAR_STATIC_BYTES (4u << 20)
int pacer_linear_static(const void *x, const void *w, float *y, int rows, int N, int K, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* PACER_H_ */
