// C-ABI entry points of the Pacer library (see include/pacer.h) and the host-side
// sequencing of the kernels.  The host only enqueues; every data-dependent
// decision (rows of a forward, stop of the draft loop, acceptance, rollback,
// end of generation) is taken by kernels from the device-resident SeqState.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <string>
#include <vector>

#include <map>

#include "common.cuh"
#include "control.cuh"
#include "fwd_kernel.cuh"
#include "gemm.cuh"

struct pacer_ctx {
    pacer_cfg cfg;
    cudaStream_t stream;
    char *ws;
    size_t ws_bytes;
    DevPtrs d;
    ModelDev model[3];
    Geom g_draft, g_mb, g_verify, g_ar, g_prefill;
    fwd::FwdBufs fb;
    int ncta;                  // blocks of the forward kernel (one per SM)
    std::map<int, fwd::Plan> plans;   // key: which * 2 + has_head
    unsigned long long *prof_stamps;
    int batch;                 // sequences of the current run
    int mode;                  // PACER_GREEDY / PACER_SAMPLE of the current run
    int prefilled;
    int64_t launches;
    cudaEvent_t ev[4];
    // one draft-and-verify step of Algorithm 1 (every draft forward and pre-verification call of the window, the
    // verify forward, the acceptance) captured once as a CUDA graph and replayed per step: the launches of a step
    // never change, all that differs from step to step lives in the device-side state.  Key: window, mode, batch.
    struct StepGraph { cudaGraph_t graph; cudaGraphExec_t exec; int64_t launches; };   // exec == NULL: seen once, not captured yet
    std::map<int64_t, StepGraph> step_graphs;
    int use_graphs;
    int32_t *fin_host;         // pinned: finished flags of the sequences, one row per step in flight
    cudaEvent_t fin_ev[8];
    std::vector<float2> rope_host[3];
    std::string err;
    size_t buf_bytes[16];
    void *buf_ptr[16];
    // kernel-level profiling (pacer_profile_begin / _end)
    int prof_on;
    std::vector<cudaEvent_t> prof_ev;      // pairs
    size_t prof_used;
    double prof_bytes;
};

static thread_local std::string g_err;

extern "C" const char *pacer_strerror(int code) {
    switch (code) {
        case PACER_OK: return "ok";
        case PACER_EINVAL: return "invalid argument";
        case PACER_ENOMEM: return "workspace too small";
        case PACER_ECUDA: return "CUDA runtime error";
        case PACER_EDEVICE: return "device-side anomaly";
        case PACER_ESTATE: return "call out of order";
        case PACER_EUNSUPPORTED: return "unsupported";
    }
    return "unknown error";
}

extern "C" const char *pacer_last_error(const pacer_ctx *ctx) { return ctx ? ctx->err.c_str() : g_err.c_str(); }

static int fail(pacer_ctx *c, int code, const std::string &msg) {
    if (c) c->err = msg;
    g_err = msg;
    return code;
}

#define CK(call)                                                                                       \
    do {                                                                                               \
        cudaError_t e_ = (call);                                                                       \
        if (e_ != cudaSuccess)                                                                         \
            return fail(c, PACER_ECUDA, std::string(#call) + ": " + cudaGetErrorString(e_));           \
    } while (0)

// ------------------------------------------------------------------ configuration

static bool model_cfg_ok(const pacer_model_cfg &m) {
    if (m.n_layers < 1 || m.d_model < 32 || m.n_heads < 1 || m.n_kv_heads < 1 || m.d_ffn < 32 || m.vocab < 2) return false;
    if (m.d_model % m.n_heads) return false;
    const int hd = m.d_model / m.n_heads;
    if (hd != 64 && hd != 128) return false;
    if (m.n_heads % m.n_kv_heads) return false;
    if (m.d_model % 64 || m.d_ffn % 64) return false;     // the weight stages are 64 k columns wide
    return true;
}

static bool cfg_ok(const pacer_cfg *c) {
    if (!c) return false;
    if (!model_cfg_ok(c->target) || !model_cfg_ok(c->draft)) return false;
    if (c->target.vocab != c->draft.vocab) return false;
    if (c->max_batch < 1 || c->max_batch > 64 || c->max_ctx < 4) return false;
    if (c->block_b < 1 || c->gamma_cap < c->block_b || c->gamma_cap % c->block_b) return false;
    if (c->criterion < 0 || c->criterion > 2) return false;
    if (c->mb_scope < 0 || c->mb_scope > 2) return false;
    if (!(c->rho > 0.f)) return false;
    if ((int64_t)c->max_batch * (c->gamma_cap + 1) > 144) return false;    // rows of one verify forward (see make_geom)
    if (c->max_batch > fwd::MAX_SEQ) return false;
    return true;
}

static pacer_model_cfg mb_cfg(const pacer_cfg &c) {
    pacer_model_cfg m = c.draft;
    m.n_layers = 1;
    return m;
}

// Rows of a forward as groups of eight-row tiles for the tensor cores: up to 32 rows one group of 1..4 tiles;
// wider forwards groups of 6 or 8 tiles (48 / 64 rows), as few padded rows as possible, three groups at most.
static Geom make_geom(int batch, int rps) {
    Geom g;
    g.batch = batch; g.rps = rps; g.rtot = batch * rps;
    const int r = g.rtot;
    if (r <= 32) { g.nt = (r + 7) / 8; g.G = 1; }
    else if (r <= 48) { g.nt = 6; g.G = 1; }
    else if (r <= 64) { g.nt = 8; g.G = 1; }
    else if (r <= 96) { g.nt = 6; g.G = 2; }
    else if (r <= 128) { g.nt = 8; g.G = 2; }
    else { g.nt = 6; g.G = 3; }                 // up to 144 rows, the most a forward takes
    g.rpad = g.G * g.nt * 8;
    return g;
}

struct Carver {
    size_t off = 0;
    size_t take(size_t bytes) {
        size_t o = off;
        off += (bytes + 255) / 256 * 256;
        return o;
    }
};

struct Layout {
    size_t st, x, y, alpha, hpend, hpend_e, draft_len, accept_len, sched_win, verify_logits, draft_logits;
    size_t row_pos, row_tok, n_rows, row_arg, row_margin, xres, att, act, hidden, part;
    size_t att_cnt, bar, abort_flag, qkv, xg, ssq, tile_top, attp, prof;
    size_t kc[3], vc[3], rope[3];
    size_t wt[3][5], wt_bytes[3][5];   // the projections re-laid for the tensor cores
    size_t kv_bytes[3], rope_bytes[3];
    size_t total;
    int rtot_max, nt_max, max_steps, d_max, f_max;
    size_t part_bytes, state_bytes;
};

static int sm_count_or_default() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
        return n;
    cudaGetLastError();
    return 148;
}

static Layout make_layout(const pacer_cfg &c) {
    Layout L;
    Carver cv;
    const pacer_model_cfg mb = mb_cfg(c);
    const pacer_model_cfg *ms[3] = {&c.target, &c.draft, &mb};
    const int B = c.max_batch, gc = c.gamma_cap, V = c.target.vocab;
    const int rps_max = gc + 1 > c.block_b + 1 ? gc + 1 : c.block_b + 1;
    L.rtot_max = std::max(B * rps_max, B * std::max(gc + 1, 128 / B));      // verify rows, prompt-chunk rows
    L.nt_max = (L.rtot_max + 7) / 8;
    const size_t RP = std::min<size_t>(fwd::MAX_ROWS, make_geom(1, std::max(L.rtot_max, 32)).rpad);   // padded rows of the widest forward
    L.max_steps = c.max_ctx;
    int d_max = 0, f_max = 0, h_max = 0, hd_max = 0, qrows_max = 0;
    for (int i = 0; i < 3; ++i) {
        const int hd = ms[i]->d_model / ms[i]->n_heads;
        d_max = std::max(d_max, ms[i]->d_model);
        f_max = std::max(f_max, ms[i]->d_ffn);
        h_max = std::max(h_max, ms[i]->n_heads);
        hd_max = std::max(hd_max, hd);
        qrows_max = std::max(qrows_max, (ms[i]->n_heads + 2 * ms[i]->n_kv_heads) * hd);
    }
    L.st = cv.take(sizeof(SeqState) * B);
    L.x = cv.take(sizeof(int32_t) * B * c.max_ctx);
    L.y = cv.take(sizeof(int32_t) * B * gc);
    L.alpha = cv.take(sizeof(float) * B * gc);
    L.hpend_e = cv.take(sizeof(int32_t) * B * (c.block_b + 1));
    L.draft_len = cv.take(sizeof(int32_t) * B * L.max_steps);
    L.accept_len = cv.take(sizeof(int32_t) * B * L.max_steps);
    L.sched_win = cv.take(sizeof(int32_t) * B * L.max_steps);
    L.row_pos = cv.take(sizeof(int32_t) * fwd::MAX_ROWS);
    L.row_tok = cv.take(sizeof(int32_t) * fwd::MAX_ROWS);
    L.n_rows = cv.take(sizeof(int32_t) * fwd::MAX_SEQ);
    L.row_arg = cv.take(sizeof(int32_t) * fwd::MAX_ROWS);
    L.row_margin = cv.take(sizeof(float) * fwd::MAX_ROWS);
    L.att_cnt = cv.take(sizeof(int32_t) * (size_t)B * h_max);
    L.bar = cv.take(sizeof(unsigned long long));
    L.abort_flag = cv.take(sizeof(int32_t) * 4);
    L.prof = cv.take(sizeof(unsigned long long) * fwd::PROF_STAMPS * fwd::PROF_BLOCKS);
    L.state_bytes = cv.off;                                   // zeroed at create
    L.hpend = cv.take(sizeof(float) * B * (c.block_b + 1) * c.draft.d_model);
    L.verify_logits = cv.take(sizeof(float) * B * (gc + 1) * V);
    L.draft_logits = cv.take(sizeof(float) * B * gc * V);
    L.d_max = d_max; L.f_max = f_max;
    L.xres = cv.take(sizeof(float) * RP * d_max);
    L.hidden = cv.take(sizeof(float) * RP * d_max);
    L.att = cv.take(sizeof(bf16) * 2 * RP * d_max);        // values, then rounding remainders
    L.act = cv.take(sizeof(bf16) * 2 * RP * f_max);
    L.qkv = cv.take(sizeof(float) * 4 * fwd::MAX_ROWS * qrows_max);     // up to four k slices, MAX_ROWS apart
    L.xg = cv.take(sizeof(bf16) * 2 * RP * d_max);
    L.ssq = cv.take(sizeof(float) * fwd::MAX_ROWS * (d_max / 16 + 1));
    L.tile_top = cv.take(sizeof(float) * 4 * fwd::MAX_ROWS * ((size_t)V / 16 + 1));
    const int rps_all = std::max(rps_max, std::max(gc + 1, 128 / B));          // rows per sequence: verify, M_B, prompt chunks
    L.attp = cv.take(sizeof(float) * (size_t)B * h_max * fwd::MAX_SPLIT * rps_all * (hd_max + 2));
    L.part_bytes = sizeof(float) * 8 * (size_t)(d_max + 16) * RP;         // up to 8 k slices of [d/16][padded rows][16]
    L.part = cv.take(L.part_bytes);
    for (int i = 0; i < 3; ++i) {
        const int hd = ms[i]->d_model / ms[i]->n_heads;
        L.kv_bytes[i] = 2 * sizeof(bf16) * (size_t)ms[i]->n_layers * B * ms[i]->n_kv_heads * c.max_ctx * hd;   // values + remainders
        L.kc[i] = cv.take(L.kv_bytes[i]);
        L.vc[i] = cv.take(L.kv_bytes[i]);
        L.rope_bytes[i] = sizeof(float2) * (size_t)c.max_ctx * (hd / 2);
        L.rope[i] = cv.take(L.rope_bytes[i]);
    }
    for (int i = 0; i < 3; ++i) {
        const pacer_model_cfg &k = *ms[i];
        const size_t hd = k.d_model / k.n_heads, qrows = (k.n_heads + 2 * (size_t)k.n_kv_heads) * hd, hh = k.n_heads * hd;
        const size_t rows16[5] = {(qrows + 15) / 16, ((size_t)k.d_model + 15) / 16, ((size_t)k.d_ffn + 7) / 8,
                                  ((size_t)k.d_model + 15) / 16, ((size_t)k.vocab + 15) / 16};       // 16-row tiles
        const size_t kdim[5] = {(size_t)k.d_model, hh, (size_t)k.d_model, (size_t)k.d_ffn, (size_t)k.d_model};
        for (int j = 0; j < 5; ++j) {
            const size_t layers = j == 4 ? (i == 2 ? 0 : 1) : (size_t)k.n_layers;
            L.wt_bytes[i][j] = layers * (kdim[j] / 64) * (2 * rows16[j]) * 1024;
            L.wt[i][j] = cv.take(L.wt_bytes[i][j]);
        }
    }
    L.total = cv.off;
    return L;
}

extern "C" size_t pacer_workspace_bytes(const pacer_cfg *cfg) {
    if (!cfg_ok(cfg)) return 0;
    return make_layout(*cfg).total;
}

static void set_geoms(pacer_ctx *c, int batch, int draft_rows = 2) {
    c->batch = batch;
    c->g_draft = make_geom(batch, draft_rows);
    c->d.sched_rows = draft_rows;
    c->g_mb = make_geom(batch, c->cfg.block_b + 1);
    c->g_verify = make_geom(batch, c->cfg.gamma_cap + 1);
    c->g_ar = make_geom(batch, 1);
    // prompt chunks: as many rows per sequence as keep the forward at 128 rows (two full row groups)
    c->g_prefill = make_geom(batch, std::max(c->cfg.gamma_cap + 1, 128 / batch));
}

extern "C" int pacer_create(const pacer_cfg *cfg, void *dev_workspace, size_t workspace_bytes, void *cuda_stream,
                            pacer_ctx **out) {
    pacer_ctx *c = nullptr;
    if (!out) return fail(nullptr, PACER_EINVAL, "out is null");
    *out = nullptr;
    if (!cfg_ok(cfg)) return fail(nullptr, PACER_EINVAL, "bad configuration");
    if (!dev_workspace || ((uintptr_t)dev_workspace & 255)) return fail(nullptr, PACER_EINVAL, "workspace null or not 256-byte aligned");
    Layout L = make_layout(*cfg);
    if (workspace_bytes < L.total) return fail(nullptr, PACER_ENOMEM, "workspace smaller than pacer_workspace_bytes");
    c = new pacer_ctx();
    c->cfg = *cfg;
    c->stream = (cudaStream_t)cuda_stream;
    c->ws = (char *)dev_workspace;
    c->ws_bytes = workspace_bytes;
    c->prefilled = 0;
    c->launches = 0;
    c->use_graphs = 1;
    if (const char *e = getenv("PACER_NO_GRAPH")) c->use_graphs = atoi(e) ? 0 : 1;
    if (c->stream == nullptr || c->stream == cudaStreamLegacy) c->use_graphs = 0;   // the legacy default stream cannot be captured
    c->prof_on = 0;
    c->prof_used = 0;
    c->prof_bytes = 0;
    DevPtrs &d = c->d;
    char *w = c->ws;
    d.st = (SeqState *)(w + L.st); d.x = (int32_t *)(w + L.x); d.y = (int32_t *)(w + L.y);
    d.alpha = (float *)(w + L.alpha); d.hpend = (float *)(w + L.hpend); d.hpend_e = (int32_t *)(w + L.hpend_e);
    d.draft_len = (int32_t *)(w + L.draft_len); d.accept_len = (int32_t *)(w + L.accept_len);
    d.sched_win = (int32_t *)(w + L.sched_win); d.sched_rows = 2;
    d.verify_logits = (float *)(w + L.verify_logits); d.draft_logits = (float *)(w + L.draft_logits);
    d.row_pos = (int32_t *)(w + L.row_pos); d.row_tok = (int32_t *)(w + L.row_tok); d.n_rows = (int32_t *)(w + L.n_rows);
    d.row_arg = (int32_t *)(w + L.row_arg); d.row_margin = (float *)(w + L.row_margin);
    d.xres = (float *)(w + L.xres); d.att = (bf16 *)(w + L.att); d.act = (bf16 *)(w + L.act);
    d.hidden = (float *)(w + L.hidden); d.part = (float *)(w + L.part);
    c->fb.qkv = (float *)(w + L.qkv); c->fb.xg = (bf16 *)(w + L.xg); c->fb.ssq = (float *)(w + L.ssq);
    c->fb.part = (float *)(w + L.part);
    c->fb.tile_top = (float *)(w + L.tile_top); c->fb.attp = (float *)(w + L.attp);
    c->fb.att_cnt = (int32_t *)(w + L.att_cnt); c->fb.bar = (unsigned long long *)(w + L.bar);
    c->fb.abort_flag = (int32_t *)(w + L.abort_flag);
    c->fb.prof = nullptr;
    c->prof_stamps = (unsigned long long *)(w + L.prof);
    c->ncta = sm_count_or_default();
    d.max_batch = cfg->max_batch; d.max_ctx = cfg->max_ctx; d.gamma_cap = cfg->gamma_cap; d.block_b = cfg->block_b;
    d.max_steps = L.max_steps; d.rho = cfg->rho; d.succ_bias = cfg->succ_bias; d.criterion = cfg->criterion;
    d.use_posemb = cfg->use_posemb;
    d.mb_scope = cfg->mb_scope;
    const pacer_model_cfg mb = mb_cfg(*cfg);
    const pacer_model_cfg *ms[3] = {&cfg->target, &cfg->draft, &mb};
    for (int i = 0; i < 3; ++i) {
        ModelDev &m = c->model[i];
        memset(&m, 0, sizeof m);
        m.cfg = *ms[i];
        m.hd = m.cfg.d_model / m.cfg.n_heads;
        m.qrows = (m.cfg.n_heads + 2 * m.cfg.n_kv_heads) * m.hd;
        m.kcache = (bf16 *)(w + L.kc[i]);
        m.vcache = (bf16 *)(w + L.vc[i]);
        m.kv_lo = L.kv_bytes[i] / (2 * sizeof(bf16));
        for (int j = 0; j < 5; ++j) m.wt[j] = L.wt_bytes[i][j] ? (const bf16 *)(w + L.wt[i][j]) : nullptr;
        m.rope = (const float2 *)(w + L.rope[i]);
        const int half = m.hd / 2;
        c->rope_host[i].resize((size_t)cfg->max_ctx * half);
        for (int p = 0; p < cfg->max_ctx; ++p)
            for (int k = 0; k < half; ++k) {
                const double ang = (double)p * pow((double)m.cfg.rope_theta, -2.0 * k / m.hd);
                c->rope_host[i][(size_t)p * half + k] = make_float2((float)cos(ang), (float)sin(ang));
            }
    }
    // buffers readable through pacer_read_buffer
    const int B = cfg->max_batch, gc = cfg->gamma_cap, V = cfg->target.vocab;
    memset(c->buf_bytes, 0, sizeof c->buf_bytes);
    auto reg = [&](int id, void *p, size_t n) { c->buf_ptr[id] = p; c->buf_bytes[id] = n; };
    reg(PACER_BUF_TOKENS, d.x, sizeof(int32_t) * B * cfg->max_ctx);
    reg(PACER_BUF_DRAFTS, d.y, sizeof(int32_t) * B * gc);
    reg(PACER_BUF_ALPHA, d.alpha, sizeof(float) * B * gc);
    reg(PACER_BUF_VERIFY_LOGITS, d.verify_logits, sizeof(float) * B * (gc + 1) * V);
    reg(PACER_BUF_DRAFT_LOGITS, d.draft_logits, sizeof(float) * B * gc * V);
    reg(PACER_BUF_HPEND, d.hpend, sizeof(float) * B * (cfg->block_b + 1) * cfg->draft.d_model);
    reg(PACER_BUF_DRAFT_LEN, d.draft_len, sizeof(int32_t) * B * L.max_steps);
    reg(PACER_BUF_ACCEPT_LEN, d.accept_len, sizeof(int32_t) * B * L.max_steps);
    reg(PACER_BUF_PHASE_NS, c->prof_stamps, sizeof(unsigned long long) * fwd::PROF_STAMPS * fwd::PROF_BLOCKS);
    for (int i = 0; i < 3; ++i) {
        reg(PACER_BUF_KCACHE_T + 2 * i, c->model[i].kcache, L.kv_bytes[i]);
        reg(PACER_BUF_VCACHE_T + 2 * i, c->model[i].vcache, L.kv_bytes[i]);
    }
    set_geoms(c, 1);
    cudaError_t e = cudaMemsetAsync(c->ws, 0, L.state_bytes, c->stream);
    for (int i = 0; i < 3 && e == cudaSuccess; ++i)
        e = cudaMemcpyAsync((void *)c->model[i].rope, c->rope_host[i].data(), L.rope_bytes[i], cudaMemcpyHostToDevice, c->stream);
    for (int i = 0; i < 4 && e == cudaSuccess; ++i) e = cudaEventCreate(&c->ev[i]);
    for (int i = 0; i < 8 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&c->fin_ev[i], cudaEventDisableTiming);
    c->fin_host = nullptr;
    if (e == cudaSuccess) e = cudaHostAlloc((void **)&c->fin_host, sizeof(int32_t) * 8 * cfg->max_batch, cudaHostAllocDefault);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) {
        std::string msg = std::string("pacer_create: ") + cudaGetErrorString(e);
        delete c;
        return fail(nullptr, PACER_ECUDA, msg);
    }
    *out = c;
    return PACER_OK;
}

extern "C" int pacer_destroy(pacer_ctx *c) {
    if (!c) return PACER_EINVAL;
    cudaStreamSynchronize(c->stream);
    for (int i = 0; i < 4; ++i) cudaEventDestroy(c->ev[i]);
    for (int i = 0; i < 8; ++i) cudaEventDestroy(c->fin_ev[i]);
    for (auto &kv : c->step_graphs)
        if (kv.second.exec) { cudaGraphExecDestroy(kv.second.exec); cudaGraphDestroy(kv.second.graph); }
    if (c->fin_host) cudaFreeHost(c->fin_host);
    for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
    delete c;
    return PACER_OK;
}

// ------------------------------------------------------------------ weights

// Re-lays one stack of [layers][N][K] row-major matrices into the order the forward kernel streams:
// [layer][K/64][atoms][8 rows][64 k], an atom being 1 KB in the 128-byte swizzle layout of a K-major tensor-core
// operand (the 16-byte chunk c of row r sits at chunk c ^ r).  Atom a holds rows 8a .. 8a+7 of W1, or, when W2 is
// given (gate/up), rows 8(a/2) .. of W1 for even a and of W2 for odd a.  Rows past N are zeros.
__global__ void k_retile(const bf16 *W1, const bf16 *W2, bf16 *out, int layers, int N, int K, int atoms) {
    const size_t total = (size_t)layers * (K / 64) * atoms * 64;          // 16-byte chunks
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int ch = (int)(i & 7), r = (int)((i >> 3) & 7);
        const size_t atom_lin = i >> 6;
        const int a = (int)(atom_lin % atoms);
        const size_t lk = atom_lin / atoms;
        const int kb = (int)(lk % (K / 64)), layer = (int)(lk / (K / 64));
        const bf16 *src = W1;
        int row = a * 8 + r;
        if (W2) { row = (a >> 1) * 8 + r; if (a & 1) src = W2; }
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (row < N) v = *reinterpret_cast<const uint4 *>(src + ((size_t)layer * N + row) * K + kb * 64 + ch * 8);
        *reinterpret_cast<uint4 *>(out + atom_lin * 512 + r * 64 + ((ch ^ r) << 3)) = v;
    }
}

extern "C" int pacer_load_weights(pacer_ctx *c, int which, const pacer_tensor *tbl, int n, const int32_t *succ) {
    if (!c || !tbl || which < 0 || which > 2 || n < 1) return fail(c, PACER_EINVAL, "pacer_load_weights: bad argument");
    ModelDev &m = c->model[which];
    const pacer_model_cfg &k = m.cfg;
    const int64_t L = k.n_layers, d = k.d_model, F = k.d_ffn, V = k.vocab, hh = (int64_t)k.n_heads * m.hd;
    struct Want { const char *name; const bf16 **slot; int64_t numel; bool needed; };
    const bool isB = which == PACER_PREVERIFY;
    Want want[] = {
        {"embed", &m.embed, V * d, !isB}, {"wqkv", &m.wqkv, L * m.qrows * d, true}, {"wo", &m.wo, L * d * hh, true},
        {"wgate", &m.wgate, L * F * d, true}, {"wup", &m.wup, L * F * d, true}, {"wdown", &m.wdown, L * d * F, true},
        {"norm1", &m.norm1, L * d, true}, {"norm2", &m.norm2, L * d, true}, {"normf", &m.normf, d, true},
        {"head", &m.head, V * d, !isB}, {"head_b", &m.head_b, 2 * d, isB},
        {"posemb", &m.posemb, (int64_t)c->cfg.gamma_cap * d, isB},
    };
    for (auto &wn : want) *wn.slot = nullptr;
    for (int i = 0; i < n; ++i) {
        if (!tbl[i].name || !tbl[i].dev_ptr) return fail(c, PACER_EINVAL, "pacer_load_weights: null entry");
        bool found = false;
        for (auto &wn : want) {
            if (strcmp(wn.name, tbl[i].name)) continue;
            found = true;
            if (!wn.needed) break;
            if (tbl[i].numel != wn.numel)
                return fail(c, PACER_EINVAL, std::string("pacer_load_weights: wrong size for ") + wn.name);
            if ((uintptr_t)tbl[i].dev_ptr & 15)
                return fail(c, PACER_EINVAL, std::string("pacer_load_weights: tensor not 16-byte aligned: ") + wn.name);
            *wn.slot = (const bf16 *)tbl[i].dev_ptr;
        }
        if (!found) return fail(c, PACER_EINVAL, std::string("pacer_load_weights: unknown tensor ") + tbl[i].name);
    }
    for (auto &wn : want)
        if (wn.needed && !*wn.slot) return fail(c, PACER_EINVAL, std::string("pacer_load_weights: missing tensor ") + wn.name);
    {
        // the library's own copy of the five projections, in streaming order (the caller's matrices are not read again)
        const int F = k.d_ffn;
        struct Job { const bf16 *w1, *w2; int j, layers, N, K, atoms; };
        const Job jobs[5] = {
            {m.wqkv, nullptr, 0, (int)L, m.qrows, (int)d, 2 * ((m.qrows + 15) / 16)},
            {m.wo, nullptr, 1, (int)L, (int)d, (int)hh, 2 * (((int)d + 15) / 16)},
            {m.wgate, m.wup, 2, (int)L, F, (int)d, 2 * ((F + 7) / 8)},
            {m.wdown, nullptr, 3, (int)L, (int)d, F, 2 * (((int)d + 15) / 16)},
            {m.head, nullptr, 4, 1, (int)V, (int)d, 2 * (((int)V + 15) / 16)},
        };
        for (const Job &jb : jobs) {
            if (!jb.w1 || !m.wt[jb.j]) continue;
            k_retile<<<148 * 8, 256, 0, c->stream>>>(jb.w1, jb.w2, const_cast<bf16 *>(m.wt[jb.j]), jb.layers, jb.N, jb.K, jb.atoms);
            CK(cudaGetLastError());
        }
    }
    m.succ = isB ? nullptr : succ;
    m.loaded = 1;
    c->plans.clear();
    for (auto &kv : c->step_graphs)
        if (kv.second.exec) { cudaGraphExecDestroy(kv.second.exec); cudaGraphDestroy(kv.second.graph); }
    c->step_graphs.clear();                    // captured launches carry the old weight pointers
    return PACER_OK;
}

// ------------------------------------------------------------------ one forward

#define LAUNCH_CHECK()                                                      \
    do {                                                                    \
        ++c->launches;                                                      \
        CK(cudaGetLastError());                                             \
    } while (0)

static double model_weight_bytes(const ModelDev &m, bool head) {
    const pacer_model_cfg &k = m.cfg;
    const double per_layer = (double)m.qrows * k.d_model + (double)k.d_model * k.n_heads * m.hd + 3.0 * k.d_model * k.d_ffn;
    return 2.0 * (k.n_layers * per_layer + (head ? (double)k.vocab * k.d_model : 0.0));
}

// Runs model `which` on the rows `kind` selects: ONE cooperative launch of the
// persistent forward kernel, which also takes the stage's decisions in its tail.
static int run_forward(pacer_ctx *c, int which, const Geom &g, int kind, int aux, bool head) {
    ModelDev &m = c->model[which];
    if (g.rtot > fwd::MAX_ROWS || g.batch > fwd::MAX_SEQ) return fail(c, PACER_EUNSUPPORTED, "too many rows or sequences in one forward");
    if (head && kind == KIND_VERIFY && g.rtot > c->ncta) return fail(c, PACER_EUNSUPPORTED, "more verify rows than blocks");
    const int key = ((which * 2 + (head ? 1 : 0)) * 16 + g.nt) * 4 + g.G;
    auto it = c->plans.find(key);
    if (it == c->plans.end()) it = c->plans.emplace(key, fwd::make_plan(m, c->d, c->fb, c->ncta, head, g)).first;
    fwd::Args a;
    a.d = c->d; a.m = m; a.g = g; a.P = it->second; a.fb = c->fb; a.kind = kind; a.aux = aux;
    a.fb.prof = (c->prof_on && c->ncta <= fwd::PROF_BLOCKS) ? c->prof_stamps : nullptr;
    const bool prof = c->prof_on && which == PACER_TARGET && c->prof_used + 2 <= c->prof_ev.size();
    if (prof) CK(cudaEventRecord(c->prof_ev[c->prof_used], c->stream));
    CK(fwd::launch(a, which, c->ncta, c->stream));
    ++c->launches;
    if (prof) {
        CK(cudaEventRecord(c->prof_ev[c->prof_used + 1], c->stream));
        c->prof_used += 2;
        c->prof_bytes += model_weight_bytes(m, head);
    }
    return PACER_OK;
}

static int need_ready(pacer_ctx *c, bool prefilled) {
    if (!c) return fail(nullptr, PACER_EINVAL, "ctx is null");
    for (int i = 0; i < 3; ++i)
        if (!c->model[i].loaded) return fail(c, PACER_ESTATE, "weights of all three models must be loaded first");
    if (prefilled && !c->prefilled) return fail(c, PACER_ESTATE, "pacer_prefill must run first");
    return PACER_OK;
}

// ------------------------------------------------------------------ stages

// windows: NULL, or host [batch][n_windows] prescribed draft windows (speculative decoding without pre-verification)
static int start_run(pacer_ctx *c, const int32_t *prompt, int batch, int n_prompt, int max_new, int gamma_max,
                     float threshold, int mode, uint64_t seed, const int32_t *windows = nullptr, int n_windows = 0) {
    const pacer_cfg &k = c->cfg;
    if (windows) {
        if (n_windows < 1 || n_windows > c->d.max_steps) return fail(c, PACER_EINVAL, "prescribed windows: bad count");
        for (int i = 0; i < batch * n_windows; ++i)
            if (windows[i] < 0 || windows[i] > k.gamma_cap) return fail(c, PACER_EINVAL, "prescribed window outside [0, gamma_cap]");
    }
    if (!prompt || batch < 1 || batch > k.max_batch || n_prompt < 1 || max_new < 1)
        return fail(c, PACER_EINVAL, "prefill: bad batch / n_prompt / max_new");
    const int gm = gamma_max / k.block_b * k.block_b;
    if (gm < k.block_b || gm > k.gamma_cap) return fail(c, PACER_EINVAL, "prefill: gamma_max outside [block_b, gamma_cap]");
    if ((int64_t)n_prompt + max_new + k.gamma_cap + 2 > k.max_ctx) return fail(c, PACER_EINVAL, "prefill: n_prompt + max_new + gamma_cap + 2 exceeds max_ctx");
    if (mode != PACER_GREEDY && mode != PACER_SAMPLE) return fail(c, PACER_EINVAL, "prefill: bad mode");
    for (int s = 0; s < batch; ++s)
        for (int i = 0; i < n_prompt; ++i)
            if (prompt[(size_t)s * n_prompt + i] < 0 || prompt[(size_t)s * n_prompt + i] >= k.target.vocab)
                return fail(c, PACER_EINVAL, "prefill: token id out of range");
    // with prescribed windows a step may draft nothing, so the draft model can fall several rows behind: its
    // forwards then take up to 16 rows per sequence (as many as fit the row limit of a forward)
    const int draft_rows = windows ? std::min(16, fwd::MAX_ROWS / batch) : 2;
    if (draft_rows < 2) return fail(c, PACER_EINVAL, "prescribed windows: batch too large");
    set_geoms(c, batch, draft_rows);
    c->mode = mode;
    std::vector<SeqState> hs(k.max_batch);
    memset(hs.data(), 0, sizeof(SeqState) * hs.size());
    for (int s = 0; s < batch; ++s) {
        SeqState &st = hs[s];
        st.P = n_prompt; st.n_prompt = n_prompt; st.max_new = max_new; st.gamma_max = gm; st.t0 = threshold;
        st.t_k = threshold; st.mode = mode; st.seed = seed; st.active = 1; st.drafting = 1;
        if (windows) {
            st.sched = 1; st.n_sched = n_windows;
            st.gamma_max = windows[(size_t)s * n_windows];
            st.drafting = st.gamma_max > 0;
        }
    }
    if (windows)
        CK(cudaMemcpy2DAsync(c->d.sched_win, sizeof(int32_t) * c->d.max_steps, windows, sizeof(int32_t) * n_windows,
                             sizeof(int32_t) * n_windows, batch, cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(c->d.st, hs.data(), sizeof(SeqState) * hs.size(), cudaMemcpyHostToDevice, c->stream));
    // arrival counters, grid barrier and abort flag start from zero (they are contiguous in the workspace)
    CK(cudaMemsetAsync(c->fb.att_cnt, 0, (char *)c->fb.abort_flag + 4 * sizeof(int32_t) - (char *)c->fb.att_cnt, c->stream));
    CK(cudaMemcpy2DAsync(c->d.x, sizeof(int32_t) * k.max_ctx, prompt, sizeof(int32_t) * n_prompt, sizeof(int32_t) * n_prompt,
                         batch, cudaMemcpyHostToDevice, c->stream));
    CK(cudaStreamSynchronize(c->stream));        // hs is a local
    return PACER_OK;
}

static int prefill_models(pacer_ctx *c, int n_prompt, bool target, bool draft_and_mb, bool mb = true) {
    const Geom &g = c->g_prefill;
    for (int c0 = 0; c0 < n_prompt - 1; c0 += g.rps) {
        int rc;
        if (target) {
            if ((rc = run_forward(c, PACER_TARGET, g, KIND_PREFILL, c0, false))) return rc;
        }
        if (draft_and_mb) {
            if ((rc = run_forward(c, PACER_DRAFT, g, KIND_PREFILL, c0, false))) return rc;
            if (mb && (rc = run_forward(c, PACER_PREVERIFY, g, KIND_PREFILL_B, c0, false))) return rc;
        }
    }
    return PACER_OK;
}

extern "C" int pacer_prefill(pacer_ctx *c, const int32_t *prompt, int batch, int n_prompt, int max_new, int gamma_max,
                             float threshold, int mode, uint64_t seed) {
    int rc = need_ready(c, false);
    if (rc) return rc;
    if ((rc = start_run(c, prompt, batch, n_prompt, max_new, gamma_max, threshold, mode, seed))) return rc;
    if ((rc = prefill_models(c, n_prompt, true, true))) return rc;
    c->prefilled = 1;
    return PACER_OK;
}

extern "C" int pacer_draft_step(pacer_ctx *c) {
    int rc = need_ready(c, true);
    if (rc) return rc;
    return run_forward(c, PACER_DRAFT, c->g_draft, KIND_DRAFT, 0, true);
}

extern "C" int pacer_preverify(pacer_ctx *c) {
    int rc = need_ready(c, true);
    if (rc) return rc;
    return run_forward(c, PACER_PREVERIFY, c->g_mb, KIND_MB, 0, false);
}

extern "C" int pacer_verify(pacer_ctx *c) {
    int rc = need_ready(c, true);
    if (rc) return rc;
    return run_forward(c, PACER_TARGET, c->g_verify, KIND_VERIFY, 0, true);
}

extern "C" int pacer_accept_rollback(pacer_ctx *c) {
    int rc = need_ready(c, true);
    if (rc) return rc;
    if (c->mode == PACER_SAMPLE) k_accept_sample<<<c->batch, ACCEPT_THREADS, 0, c->stream>>>(c->d, c->g_verify, c->cfg.target.vocab);
    else k_accept_greedy<<<1, 64, 0, c->stream>>>(c->d, c->g_verify);
    LAUNCH_CHECK();
    return PACER_OK;
}

// After a synchronisation: the device status word.  A bounded wait inside a kernel that ran out leaves its code
// there (and the block, warp and detail of the first such wait); the kernels then fall through to their end, and
// every [sync] entry point reports PACER_EDEVICE until the next run resets the word.
static int device_status(pacer_ctx *c) {
    int32_t aborted[4] = {0, 0, 0, 0};
    CK(cudaMemcpy(aborted, c->fb.abort_flag, sizeof aborted, cudaMemcpyDeviceToHost));
    if (aborted[0])
        return fail(c, PACER_EDEVICE, "a bounded wait inside the forward kernel ran out (wait code " + std::to_string(aborted[0]) +
                                          ", block " + std::to_string(aborted[1]) + ", warp " + std::to_string(aborted[2]) +
                                          ", detail " + std::to_string(aborted[3]) + ")");
    return PACER_OK;
}

extern "C" int pacer_debug_set_device_status(pacer_ctx *c, int code, int block, int warp, int detail) {
    if (!c) return fail(nullptr, PACER_EINVAL, "ctx is null");
    const int32_t v[4] = {code, block, warp, detail};
    CK(cudaMemcpyAsync(c->fb.abort_flag, v, sizeof v, cudaMemcpyHostToDevice, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return PACER_OK;
}

extern "C" int pacer_read_state(pacer_ctx *c, pacer_seq_state *out, int batch) {
    if (!c || !out || batch < 1 || batch > c->cfg.max_batch) return fail(c, PACER_EINVAL, "pacer_read_state: bad argument");
    std::vector<SeqState> hs(batch);
    CK(cudaMemcpyAsync(hs.data(), c->d.st, sizeof(SeqState) * batch, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    const int status = device_status(c);
    for (int s = 0; s < batch; ++s) {
        const SeqState &a = hs[s];
        pacer_seq_state &o = out[s];
        o.P = a.P; o.len_T = a.len_T; o.len_D = a.len_D; o.len_B = a.len_B; o.gamma = a.gamma; o.k_round = a.k_round;
        o.t_k = a.t_k; o.drafting = a.drafting; o.finished = a.finished; o.n_steps = a.n_steps; o.last_n = a.last_n;
        o.last_next = a.last_next; o.n_pend = a.n_pend; o.err = a.err; o.n_draft_fwd = a.n_draft_fwd;
        o.n_mb_calls = a.n_mb_calls; o.n_target_fwd = a.n_target_fwd;
    }
    return status;
}

extern "C" int pacer_read_buffer(pacer_ctx *c, int which, void *host_dst, size_t bytes) {
    if (!c || !host_dst || which < 0 || which >= 16 || !c->buf_bytes[which]) return fail(c, PACER_EINVAL, "pacer_read_buffer: bad buffer");
    if (bytes > c->buf_bytes[which]) return fail(c, PACER_EINVAL, "pacer_read_buffer: more bytes than the buffer holds");
    CK(cudaMemcpyAsync(host_dst, c->buf_ptr[which], bytes, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return device_status(c);
}

extern "C" int pacer_profile_begin(pacer_ctx *c) {
    if (!c) return fail(nullptr, PACER_EINVAL, "ctx is null");
    while (c->prof_ev.size() < 8192) {
        cudaEvent_t e;
        CK(cudaEventCreate(&e));
        c->prof_ev.push_back(e);
    }
    c->prof_used = 0;
    c->prof_bytes = 0;
    c->prof_on = 1;
    return PACER_OK;
}

extern "C" int pacer_profile_end(pacer_ctx *c, double *gemm_ms, double *gemm_weight_bytes, int64_t *gemm_launches) {
    if (!c || !gemm_ms || !gemm_weight_bytes || !gemm_launches) return fail(c, PACER_EINVAL, "pacer_profile_end: null argument");
    c->prof_on = 0;
    CK(cudaStreamSynchronize(c->stream));
    double ms = 0;
    for (size_t i = 0; i + 1 < c->prof_used; i += 2) {
        float t;
        CK(cudaEventElapsedTime(&t, c->prof_ev[i], c->prof_ev[i + 1]));
        ms += t;
    }
    *gemm_ms = ms;
    *gemm_weight_bytes = c->prof_bytes;
    *gemm_launches = (int64_t)(c->prof_used / 2);
    return PACER_OK;
}

// ------------------------------------------------------------------ whole loops

// The verify forward of a whole-loop run: greedy runs take the acceptance in the forward's tail, sampling
// runs in the acceptance kernel that follows.
static int enqueue_verify_accept(pacer_ctx *c) {
    int rc = need_ready(c, true);
    if (rc) return rc;
    if (c->mode == PACER_GREEDY) return run_forward(c, PACER_TARGET, c->g_verify, KIND_VERIFY, 1, true);
    if ((rc = run_forward(c, PACER_TARGET, c->g_verify, KIND_VERIFY, 0, true))) return rc;
    return pacer_accept_rollback(c);
}

// One draft-and-verify step of Algorithm 1.  Forwards of sequences that have stopped drafting are no-ops.
static int enqueue_step(pacer_ctx *c, int gamma_max) {
    int rc;
    const int b = c->cfg.block_b;
    for (int blk = 0; blk < gamma_max / b; ++blk) {
        for (int i = 0; i < b; ++i)
            if ((rc = pacer_draft_step(c))) return rc;
        if ((rc = pacer_preverify(c))) return rc;
    }
    return enqueue_verify_accept(c);
}

// One step of Algorithm 1 as a graph launch (captured on first use).  Falls back to plain launches while the
// per-launch profiling is on (its event records must stay outside a graph).
static int launch_step(pacer_ctx *c, int gamma_max) {
    if (!c->use_graphs || c->prof_on) return enqueue_step(c, gamma_max);
    const int64_t key = ((int64_t)gamma_max * 4 + c->mode) * 256 + c->batch;
    auto it = c->step_graphs.find(key);
    if (it == c->step_graphs.end()) {
        // the first step of a kind runs as plain launches (they set the kernels' shared-memory attributes, which
        // must not happen inside a capture); the second one is captured
        c->step_graphs.emplace(key, pacer_ctx::StepGraph{});
        return enqueue_step(c, gamma_max);
    }
    if (!it->second.exec) {
        pacer_ctx::StepGraph sg{};
        const int64_t before = c->launches;
        CK(cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
        const int rc = enqueue_step(c, gamma_max);
        cudaError_t e = cudaStreamEndCapture(c->stream, &sg.graph);
        sg.launches = c->launches - before;
        c->launches = before;
        if (rc) { if (e == cudaSuccess && sg.graph) cudaGraphDestroy(sg.graph); return rc; }
        CK(e);
        CK(cudaGraphInstantiate(&sg.exec, sg.graph, 0));
        it->second = sg;
    }
    CK(cudaGraphLaunch(it->second.exec, c->stream));
    c->launches += it->second.launches;
    return PACER_OK;
}

// Enqueues steps until every sequence is finished.  The end of generation is decided on the device; the host only
// learns of it, without ever waiting for the step it has just enqueued: after each step the finished flags are
// copied to pinned memory behind an event, and the host looks at the flags of the step it enqueued RUN_AHEAD steps
// ago.  Steps enqueued after the last real one are no-ops on the device.
template <class Enqueue>
static int run_steps(pacer_ctx *c, int batch, int max_steps, Enqueue enqueue) {
    constexpr int RUN_AHEAD = 2, SLOTS = 8;
    for (int step = 0; step < max_steps; ++step) {
        int rc = enqueue(step);
        if (rc) return rc;
        const int slot = step % SLOTS;
        CK(cudaMemcpy2DAsync(c->fin_host + (size_t)slot * c->cfg.max_batch, sizeof(int32_t), &c->d.st[0].finished, sizeof(SeqState),
                             sizeof(int32_t), batch, cudaMemcpyDeviceToHost, c->stream));
        CK(cudaEventRecord(c->fin_ev[slot], c->stream));
        if (step >= RUN_AHEAD) {
            const int seen = (step - RUN_AHEAD) % SLOTS;
            CK(cudaEventSynchronize(c->fin_ev[seen]));
            bool all = true;
            for (int q = 0; q < batch; ++q) all = all && c->fin_host[(size_t)seen * c->cfg.max_batch + q];
            if (all) break;
        }
    }
    return PACER_OK;
}

static int collect(pacer_ctx *c, int batch, int max_new, int n_prompt, int32_t *out_tokens, int32_t *out_n_steps,
                   int32_t *out_draft_len, int32_t *out_accept_len, pacer_stats *stats, int64_t launches0) {
    const pacer_cfg &k = c->cfg;
    std::vector<SeqState> hs(batch);
    CK(cudaMemcpyAsync(hs.data(), c->d.st, sizeof(SeqState) * batch, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpy2DAsync(out_tokens, sizeof(int32_t) * max_new, c->d.x + n_prompt, sizeof(int32_t) * k.max_ctx,
                         sizeof(int32_t) * max_new, batch, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (int rc = device_status(c)) return rc;
    int64_t nd = 0, nm = 0, nt = 0, ns = 0, ng = 0;
    for (int s = 0; s < batch; ++s) {
        const SeqState &a = hs[s];
        nd += a.n_draft_fwd; nm += a.n_mb_calls; nt += a.n_target_fwd; ns += a.n_steps; ng += a.P - a.n_prompt;
        if (out_n_steps) out_n_steps[s] = a.n_steps;
        if (out_draft_len && out_accept_len) {
            for (int i = 0; i < max_new; ++i) out_draft_len[(size_t)s * max_new + i] = out_accept_len[(size_t)s * max_new + i] = -1;
            const int n = a.n_steps < max_new ? a.n_steps : max_new;
            if (n > 0) {
                CK(cudaMemcpy(out_draft_len + (size_t)s * max_new, c->d.draft_len + (size_t)s * c->d.max_steps, sizeof(int32_t) * n, cudaMemcpyDeviceToHost));
                CK(cudaMemcpy(out_accept_len + (size_t)s * max_new, c->d.accept_len + (size_t)s * c->d.max_steps, sizeof(int32_t) * n, cudaMemcpyDeviceToHost));
            }
        }
    }
    if (stats) {
        stats->n_draft_fwd = nd; stats->n_mb_calls = nm; stats->n_target_fwd = nt; stats->n_steps = ns; stats->n_generated = ng;
        stats->n_kernel_launches = c->launches - launches0;
        CK(cudaEventElapsedTime(&stats->ms_prefill, c->ev[0], c->ev[1]));
        CK(cudaEventElapsedTime(&stats->ms_decode, c->ev[1], c->ev[2]));
    }
    return PACER_OK;
}

extern "C" int pacer_generate(pacer_ctx *c, const int32_t *prompt, int batch, int n_prompt, int max_new, int gamma_max,
                              float threshold, int mode, uint64_t seed, int32_t *out_tokens, int32_t *out_n_steps,
                              int32_t *out_draft_len, int32_t *out_accept_len, pacer_stats *stats) {
    int rc = need_ready(c, false);
    if (rc) return rc;
    if (!out_tokens) return fail(c, PACER_EINVAL, "pacer_generate: out_tokens is null");
    if ((rc = start_run(c, prompt, batch, n_prompt, max_new, gamma_max, threshold, mode, seed))) return rc;
    CK(cudaEventRecord(c->ev[0], c->stream));
    if ((rc = prefill_models(c, n_prompt, true, true))) return rc;
    c->prefilled = 1;
    CK(cudaEventRecord(c->ev[1], c->stream));
    const int64_t launches0 = c->launches;
    const int gm = gamma_max / c->cfg.block_b * c->cfg.block_b;
    if ((rc = run_steps(c, batch, max_new, [&](int) { return launch_step(c, gm); }))) return rc;
    CK(cudaEventRecord(c->ev[2], c->stream));
    return collect(c, batch, max_new, n_prompt, out_tokens, out_n_steps, out_draft_len, out_accept_len, stats, launches0);
}

extern "C" int pacer_generate_sched(pacer_ctx *c, const int32_t *prompt, int batch, int n_prompt, int max_new,
                                    const int32_t *windows, int n_windows, int mode, uint64_t seed, int32_t *out_tokens,
                                    int32_t *out_n_steps, int32_t *out_draft_len, int32_t *out_accept_len, pacer_stats *stats) {
    int rc = need_ready(c, false);
    if (rc) return rc;
    if (!out_tokens || !windows) return fail(c, PACER_EINVAL, "pacer_generate_sched: out_tokens or windows is null");
    if ((rc = start_run(c, prompt, batch, n_prompt, max_new, c->cfg.gamma_cap, -1.f, mode, seed, windows, n_windows))) return rc;
    CK(cudaEventRecord(c->ev[0], c->stream));
    if ((rc = prefill_models(c, n_prompt, true, true, false))) return rc;
    c->prefilled = 1;
    CK(cudaEventRecord(c->ev[1], c->stream));
    const int64_t launches0 = c->launches;
    rc = run_steps(c, batch, max_new, [&](int step) {
        int w = 1;                        // (a backlog of the draft model can turn a window of 0 into 1 on the device)
        for (int q = 0; q < batch; ++q) w = std::max(w, (int)windows[(size_t)q * n_windows + std::min(step, n_windows - 1)]);
        for (int i = 0; i < w; ++i) {
            int r = pacer_draft_step(c);
            if (r) return r;
        }
        return enqueue_verify_accept(c);
    });
    if (rc) return rc;
    CK(cudaEventRecord(c->ev[2], c->stream));
    return collect(c, batch, max_new, n_prompt, out_tokens, out_n_steps, out_draft_len, out_accept_len, stats, launches0);
}

extern "C" int pacer_generate_ar(pacer_ctx *c, const int32_t *prompt, int batch, int n_prompt, int max_new, int mode,
                                 uint64_t seed, int32_t *out_tokens, pacer_stats *stats) {
    int rc = need_ready(c, false);
    if (rc) return rc;
    if (!out_tokens) return fail(c, PACER_EINVAL, "pacer_generate_ar: out_tokens is null");
    if ((rc = start_run(c, prompt, batch, n_prompt, max_new, c->cfg.block_b, -1.f, mode, seed))) return rc;
    CK(cudaEventRecord(c->ev[0], c->stream));
    if ((rc = prefill_models(c, n_prompt, true, false))) return rc;
    c->prefilled = 0;                     // draft and M_B caches were not filled
    CK(cudaEventRecord(c->ev[1], c->stream));
    const int64_t launches0 = c->launches;
    for (int i = 0; i < max_new; ++i) {
        if ((rc = run_forward(c, PACER_TARGET, c->g_ar, KIND_AR, 0, true))) return rc;
    }
    CK(cudaEventRecord(c->ev[2], c->stream));
    return collect(c, batch, max_new, n_prompt, out_tokens, nullptr, nullptr, nullptr, stats, launches0);
}

// ------------------------------------------------------------------ stand-alone product

__global__ void k_to_frag(const bf16 *x, bf16 *xf, int rows, int K, int nt) {
    const int r = blockIdx.y, k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    xf[xfrag_index(r, k, nt)] = r < rows ? x[(size_t)r * K + k] : __float2bfloat16(0.f);
}

__global__ void k_sum_part(const float *part, float *y, int rows, int N, int S, int rpad) {
    const int r = blockIdx.y, n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= N || r >= rows) return;
    float v = 0.f;
    for (int s = 0; s < S; ++s) v += part[((size_t)s * rpad + r) * N + n];
    y[(size_t)r * N + n] = v;
}

extern "C" size_t pacer_linear_scratch_bytes(int rows, int N, int K) {
    if (rows < 1 || rows > 32 || N < 1 || K < 32 || K % 32) return 0;
    const int nt = (rows + 7) / 8;
    GemmPlan p = gemm_plan(N, K, nt);
    size_t xf = ((size_t)nt * 8 * K * sizeof(bf16) + 255) / 256 * 256;
    return xf + (size_t)p.S * nt * 8 * N * sizeof(float);
}

extern "C" int pacer_linear(const void *x, const void *w, float *y, int rows, int N, int K, void *scratch,
                            size_t scratch_bytes, void *cuda_stream) {
    pacer_ctx *c = nullptr;
    const size_t need = pacer_linear_scratch_bytes(rows, N, K);
    if (!x || !w || !y || !scratch || need == 0) return fail(nullptr, PACER_EINVAL, "pacer_linear: bad argument");
    if (scratch_bytes < need) return fail(nullptr, PACER_ENOMEM, "pacer_linear: scratch too small");
    if (((uintptr_t)w & 15) || ((uintptr_t)scratch & 255)) return fail(nullptr, PACER_EINVAL, "pacer_linear: misaligned pointer");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int nt = (rows + 7) / 8;
    bf16 *xf = (bf16 *)scratch;
    float *part = (float *)((char *)scratch + ((size_t)nt * 8 * K * sizeof(bf16) + 255) / 256 * 256);
    k_to_frag<<<dim3((K + 255) / 256, nt * 8), 256, 0, st>>>((const bf16 *)x, xf, rows, K, nt);
    CK(cudaGetLastError());
    GemmPlan p;
    CK(gemm_run(xf, nt, (const bf16 *)w, nullptr, 0, N, K, part, nullptr, 0, st, &p, nullptr));
    k_sum_part<<<dim3((N + 255) / 256, rows), 256, 0, st>>>(part, y, rows, N, p.S, nt * 8);
    CK(cudaGetLastError());
    return PACER_OK;
}

// ------------------------------------------------------------------ product without caller scratch

// Scratch of pacer_linear_static.  In host code this name is only a handle for
// cudaGetSymbolAddress; the device address is looked up once per device.
static __device__ __align__(256) unsigned char g_linear_static_scratch[PACER_LINEAR_STATIC_BYTES];
static void *g_linear_static_ptr[64];

extern "C" int pacer_linear_static(const void *x, const void *w, float *y, int rows, int N, int K, void *cuda_stream) {
    pacer_ctx *c = nullptr;
    const size_t need = pacer_linear_scratch_bytes(rows, N, K);
    if (!x || !w || !y || need == 0) return fail(nullptr, PACER_EINVAL, "pacer_linear_static: bad argument");
    if (need > (size_t)PACER_LINEAR_STATIC_BYTES)
        return fail(nullptr, PACER_ENOMEM, "pacer_linear_static: shape needs more than PACER_LINEAR_STATIC_BYTES of scratch");
    int dev = -1;
    CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return fail(nullptr, PACER_EUNSUPPORTED, "pacer_linear_static: device index out of range");
    if (!g_linear_static_ptr[dev]) {
        void *p = nullptr;
        CK(cudaGetSymbolAddress(&p, g_linear_static_scratch));
        if (!p) return fail(nullptr, PACER_ECUDA, "pacer_linear_static: no device address for the scratch array");
        g_linear_static_ptr[dev] = p;
    }
    return pacer_linear(x, w, y, rows, N, K, g_linear_static_ptr[dev], (size_t)PACER_LINEAR_STATIC_BYTES, cuda_stream);
}
