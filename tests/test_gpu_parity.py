"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the
same seeded inputs.  Tolerances: logits 2e-2 absolute (bf16 weights and GEMM
inputs, fp32 accumulate, against an fp64 oracle reading the same bf16 weights);
tokens, draft lengths and accept lengths bit-exact, asserted only after checking
that the oracle's deciding margins exceed the tolerance."""
import numpy as np
import pytest
import torch

from oracle import pacer_oracle as orc
from paper_2602_01274_b200 import synth
from tests.common import oracle_models

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2
ALPHA_TOL = 2e-3


def _binding():
    from paper_2602_01274_b200 import binding
    return binding


def _bf16_np(t):
    return t.detach().float().cpu().double().numpy()


# ------------------------------------------------------------------ the skinny GEMM alone

@pytest.mark.parametrize("rows,N,K", [
    (1, 256, 128), (2, 2304, 768), (5, 768, 3072), (9, 4096, 256), (17, 1000, 512), (3, 24, 64),
    (17, 12288, 4096), (17, 4096, 11008), (25, 9216, 7168), (32, 4096, 4096), (8, 32000, 768),
])
def test_linear_matches_oracle(rows, N, K):
    b = _binding()
    dev = "cuda:0"
    w = synth.normal_bf16(3, 11, (N, K), std=0.02, device=dev)
    x = synth.normal_bf16(4, 12, (rows, K), std=1.0, device=dev)
    y = b.pacer_linear(x, w).cpu().double().numpy()
    rng = np.random.default_rng(N + K)
    cols = np.unique(np.concatenate([np.arange(min(N, 24)), np.arange(max(0, N - 24), N),
                                     rng.integers(0, N, size=min(N, 200))]))
    ref = orc.linear(w[torch.as_tensor(cols, device=dev)].cpu(), _bf16_np(x))
    err = np.abs(y[:, cols] - ref).max()
    assert err < 2e-4 * max(1.0, np.abs(ref).max()), err


def test_linear_rejects_bad_shapes():
    b = _binding()
    x = torch.zeros(33, 64, dtype=torch.bfloat16, device="cuda:0")
    w = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(b.PacerError):
        b.pacer_linear(x, w)                      # more than 32 rows
    with pytest.raises(b.PacerError):
        b.pacer_linear(x[:4, :48].contiguous(), w[:, :48].contiguous())   # K not a multiple of 32


# ------------------------------------------------------------------ the loop on the tiny pair

@pytest.fixture(scope="module")
def tiny():
    b = _binding()
    cfg = synth.CONFIGS["tiny"]
    pair_gpu = synth.make_pair(cfg, seed=0, device="cuda:0")
    pair_cpu = {k: ({n: t.cpu() for n, t in v.items()} if isinstance(v, dict) else v.cpu()) for k, v in pair_gpu.items()}
    T, D, B = oracle_models(cfg, pair_cpu)
    max_ctx = cfg.n_prompt + cfg.max_new + cfg.gamma_cap + 2
    ccfg = b.make_cfg(cfg.target, cfg.draft, 1, max_ctx, cfg.gamma_cap, cfg.block_b, cfg.rho, 0, cfg.succ_bias)
    ctx = b.Context(ccfg)
    b.load_pair(ctx, pair_gpu)
    prompt = synth.make_prompts(cfg.target.vocab, 1, cfg.n_prompt, seed=0)[0].numpy()
    yield dict(cfg=cfg, ctx=ctx, T=T, D=D, B=B, prompt=prompt, max_ctx=max_ctx, b=b)
    ctx.close()


def _gpu_cache(t, which, b):
    """(k, v) float64 [L][max_ctx][Hkv*hd] of sequence 0 from the device cache."""
    ctx, cfg = t["ctx"], t["cfg"]
    shape = (cfg.target, cfg.draft, synth.preverify_shape(cfg.draft))[which]
    L, Hkv, hd = shape.n_layers, shape.n_kv_heads, shape.head_dim
    n = L * 1 * Hkv * t["max_ctx"] * hd
    out = []
    for buf in (b.BUF_KCACHE_T + 2 * which, b.BUF_VCACHE_T + 2 * which):
        raw = ctx.pacer_read_buffer(buf, np.int16, n)
        a = torch.from_numpy(raw.copy()).view(torch.bfloat16).double().numpy().reshape(L, Hkv, t["max_ctx"], hd)
        out.append(a.transpose(0, 2, 1, 3).reshape(L, t["max_ctx"], Hkv * hd))
    return out


def test_stage_by_stage_against_oracle(tiny):
    """Prefill, then three whole steps, comparing after every C-ABI call."""
    b, cfg, ctx = tiny["b"], tiny["cfg"], tiny["ctx"]
    V, gc, bb = cfg.target.vocab, cfg.gamma_cap, cfg.block_b
    o = orc.Pacer(tiny["T"], tiny["D"], tiny["B"], tiny["max_ctx"], b=bb, gamma_cap=gc, t0=0.49, rho=cfg.rho)
    o.prefill(tiny["prompt"])
    ctx.pacer_prefill(tiny["prompt"], cfg.max_new, cfg.gamma_max, 0.49)
    st = ctx.pacer_read_state()[0]
    assert (st["P"], st["len_T"], st["len_D"], st["len_B"]) == (o.P, o.cache_len(0), o.cache_len(1), o.cache_len(2))
    for which in range(3):
        ko, vo = o.cache_kv(which)
        kg, vg = _gpu_cache(tiny, which, b)
        n = o.cache_len(which)
        # bf16 storage of values of size ~1: half an ulp is 2^-9 relative
        assert np.abs(kg[:, :n] - ko[:, :n]).max() < 2e-2
        assert np.abs(vg[:, :n] - vo[:, :n]).max() < 2e-2
    for step in range(3):
        while o.drafting:
            for i in range(bb):
                ctx.pacer_draft_step()
            o.draft_block()
            st = ctx.pacer_read_state()[0]
            assert (st["gamma"], st["len_D"], st["n_pend"]) == (o.gamma, o.cache_len(1), o.n_pend)
            y = ctx.pacer_read_buffer(b.BUF_DRAFTS, np.int32, gc)[: o.gamma]
            np.testing.assert_array_equal(y, o.y())
            ql = ctx.pacer_read_buffer(b.BUF_DRAFT_LOGITS, np.float32, gc * V).reshape(gc, V)[: o.gamma]
            assert np.abs(ql - o.qlogits(o.gamma)).max() < LOGIT_TOL
            hp = ctx.pacer_read_buffer(b.BUF_HPEND, np.float32, (bb + 1) * cfg.draft.d_model)
            hp = hp.reshape(bb + 1, -1)[: o.n_pend]
            assert np.abs(hp - o.hpend()).max() < LOGIT_TOL
            ctx.pacer_preverify()
            o.preverify()
            st = ctx.pacer_read_state()[0]
            al = ctx.pacer_read_buffer(b.BUF_ALPHA, np.float32, gc)[: o.gamma]
            assert np.abs(al - o.alpha()).max() < ALPHA_TOL
            assert st["len_B"] == o.cache_len(2) and st["n_pend"] == 0
            assert st["drafting"] == o.drafting and st["t_k"] == np.float32(o.t_k)
        ctx.pacer_verify()
        o.verify()
        rows = o.gamma + 1
        pl = ctx.pacer_read_buffer(b.BUF_VERIFY_LOGITS, np.float32, (gc + 1) * V).reshape(gc + 1, V)[:rows]
        assert np.abs(pl - o.plogits(rows)).max() < LOGIT_TOL
        ctx.pacer_accept_rollback()
        n = o.accept()
        st = ctx.pacer_read_state()[0]
        assert (st["last_n"], st["last_next"], st["P"]) == (n, o.last_next, o.P)
        assert (st["len_T"], st["len_D"], st["len_B"]) == (o.cache_len(0), o.cache_len(1), o.cache_len(2))
        assert (st["gamma"], st["drafting"], st["n_steps"]) == (0, 1, step + 1)
        x = ctx.pacer_read_buffer(b.BUF_TOKENS, np.int32, tiny["max_ctx"])[: o.P]
        np.testing.assert_array_equal(x, o.x())


@pytest.mark.parametrize("t0", [-1.0, 0.46, 0.49, 0.7])
def test_generate_matches_oracle_token_for_token(tiny, t0):
    b, cfg, ctx = tiny["b"], tiny["cfg"], tiny["ctx"]
    o = orc.Pacer(tiny["T"], tiny["D"], tiny["B"], tiny["max_ctx"], b=cfg.block_b, gamma_cap=cfg.gamma_cap, t0=t0,
                  rho=cfg.rho)
    out_o, dl_o, al_o, st_o = o.generate(tiny["prompt"], cfg.max_new)
    # the comparison is exact only where the oracle's decisions are not within tolerance of a tie
    assert st_o["min_margin_target"] > 2 * LOGIT_TOL and st_o["min_margin_draft"] > 2 * LOGIT_TOL
    if t0 >= 0:
        assert st_o["min_margin_stop"] > ALPHA_TOL, st_o["min_margin_stop"]
    tok, ns, dl, al, st = ctx.pacer_generate(tiny["prompt"], cfg.max_new, cfg.gamma_max, t0)
    np.testing.assert_array_equal(tok[0], out_o)
    assert ns[0] == len(dl_o)
    np.testing.assert_array_equal(dl[0, : ns[0]], dl_o)
    np.testing.assert_array_equal(al[0, : ns[0]], al_o)
    assert (dl[0, ns[0]:] == -1).all() and (al[0, ns[0]:] == -1).all()
    assert st["n_draft_fwd"] == st_o["n_draft_fwd"] and st["n_target_fwd"] == st_o["n_target_fwd"]
    assert st["n_mb_calls"] == st_o["n_mb_calls"] and st["n_steps"] == st_o["n_steps"]
    assert st["n_kernel_launches"] > 0


def test_gpu_autoregressive_equals_oracle_and_speculative_is_lossless(tiny):
    cfg, ctx = tiny["cfg"], tiny["ctx"]
    ar_o, margin = orc.generate_ar(tiny["T"], tiny["prompt"], cfg.max_new)
    assert margin > 2 * LOGIT_TOL
    ar_g, st = ctx.pacer_generate_ar(tiny["prompt"], cfg.max_new)
    np.testing.assert_array_equal(ar_g[0], ar_o)
    assert st["n_target_fwd"] == cfg.max_new
    for t0 in (-1.0, 0.49):
        tok, *_ = ctx.pacer_generate(tiny["prompt"], cfg.max_new, cfg.gamma_max, t0)
        np.testing.assert_array_equal(tok[0], ar_g[0])


@pytest.mark.parametrize("n_prompt,max_new,gamma_max", [(1, 5, 4), (2, 1, 8), (7, 9, 4), (64, 3, 8)])
def test_edge_lengths(tiny, n_prompt, max_new, gamma_max):
    cfg, ctx = tiny["cfg"], tiny["ctx"]
    prompt = tiny["prompt"][:n_prompt]
    o = orc.Pacer(tiny["T"], tiny["D"], tiny["B"], tiny["max_ctx"], b=cfg.block_b, gamma_cap=gamma_max, t0=0.49,
                  rho=cfg.rho)
    out_o, dl_o, al_o, st_o = o.generate(prompt, max_new)
    assert st_o["min_margin_stop"] > ALPHA_TOL
    tok, ns, dl, al, _ = ctx.pacer_generate(prompt, max_new, gamma_max, 0.49)
    np.testing.assert_array_equal(tok[0], out_o)
    np.testing.assert_array_equal(dl[0, : ns[0]], dl_o[:max_new])
    np.testing.assert_array_equal(al[0, : ns[0]], al_o[:max_new])


def test_bad_arguments_are_refused_before_any_launch(tiny):
    b, cfg, ctx = tiny["b"], tiny["cfg"], tiny["ctx"]
    with pytest.raises(b.PacerError):
        ctx.pacer_generate(tiny["prompt"], cfg.max_new, 2, 0.5)                 # gamma_max < block_b
    with pytest.raises(b.PacerError):
        ctx.pacer_generate(tiny["prompt"], 10 * cfg.max_new, cfg.gamma_max, 0.5)  # does not fit max_ctx
    bad = tiny["prompt"].copy()
    bad[3] = cfg.target.vocab
    with pytest.raises(b.PacerError):
        ctx.pacer_generate(bad, cfg.max_new, cfg.gamma_max, 0.5)                # token id out of range
    bcfg = b.make_cfg(cfg.target, cfg.draft, 1, 64, 6, 4)                       # gamma_cap not a multiple of b
    assert b.pacer_workspace_bytes(bcfg) == 0
