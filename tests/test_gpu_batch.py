"""Batched decoding: independent sequences share the forwards, each with its own adaptive draft length, accept
length and cache rollback (a sequence that stopped drafting idles until the others stop; a finished sequence
idles until the batch is done).  Every sequence must come out exactly as when it is decoded alone."""
import numpy as np
import pytest
import torch

from oracle import pacer_oracle as orc
from paper_2602_01274_b200 import synth
from tests.common import oracle_models

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2
ALPHA_TOL = 2e-3


@pytest.fixture(scope="module")
def tiny3():
    from paper_2602_01274_b200 import binding as b
    cfg = synth.CONFIGS["tiny"]
    pair_gpu = synth.make_pair(cfg, seed=0, device="cuda:0")
    pair_cpu = {k: ({n: t.cpu() for n, t in v.items()} if isinstance(v, dict) else v.cpu()) for k, v in pair_gpu.items()}
    T, D, B = oracle_models(cfg, pair_cpu)
    max_ctx = cfg.n_prompt + cfg.max_new + cfg.gamma_cap + 2
    ctx = b.Context(b.make_cfg(cfg.target, cfg.draft, 3, max_ctx, cfg.gamma_cap, cfg.block_b, cfg.rho, 0, cfg.succ_bias))
    b.load_pair(ctx, pair_gpu)
    prompts = synth.make_prompts(cfg.target.vocab, 3, cfg.n_prompt, seed=4).numpy()
    yield dict(cfg=cfg, ctx=ctx, T=T, D=D, B=B, prompts=prompts, max_ctx=max_ctx, b=b)
    ctx.close()


@pytest.mark.parametrize("t0", [-1.0, 0.505])
def test_batch_of_three_equals_three_single_runs(tiny3, t0):
    cfg, ctx = tiny3["cfg"], tiny3["ctx"]
    tok, ns, dl, al, st = ctx.pacer_generate(tiny3["prompts"], cfg.max_new, cfg.gamma_max, t0)
    steps = set()
    for s in range(3):
        o = orc.Pacer(tiny3["T"], tiny3["D"], tiny3["B"], tiny3["max_ctx"], b=cfg.block_b, gamma_cap=cfg.gamma_cap,
                      t0=t0, rho=cfg.rho)
        out_o, dl_o, al_o, st_o = o.generate(tiny3["prompts"][s], cfg.max_new)
        assert st_o["min_margin_target"] > 2 * LOGIT_TOL and st_o["min_margin_draft"] > 2 * LOGIT_TOL
        if t0 >= 0:
            assert st_o["min_margin_stop"] > ALPHA_TOL
        np.testing.assert_array_equal(tok[s], out_o)
        assert ns[s] == len(dl_o)
        np.testing.assert_array_equal(dl[s, : ns[s]], dl_o)
        np.testing.assert_array_equal(al[s, : ns[s]], al_o)
        steps.add(int(ns[s]))
    assert len(steps) > 1, "the sequences should need different numbers of steps (ragged progress)"
    one, ns1, *_ = ctx.pacer_generate(tiny3["prompts"][1], cfg.max_new, cfg.gamma_max, t0)   # the same context, batch 1
    np.testing.assert_array_equal(one[0], tok[1])


def test_batched_autoregressive(tiny3):
    cfg, ctx = tiny3["cfg"], tiny3["ctx"]
    tok, _ = ctx.pacer_generate_ar(tiny3["prompts"], 24)
    for s in range(3):
        out_o, margin = orc.generate_ar(tiny3["T"], tiny3["prompts"][s], 24)
        assert margin > 2 * LOGIT_TOL
        np.testing.assert_array_equal(tok[s], out_o)


# ------------------------------------------------------------------ wide forwards: more than 32 rows

WIDE = {
    # 8 sequences x 9 verify rows = 72 rows (two row groups of 48), M_B forwards of 40 rows (one group of 48)
    "tiny_b8": (synth.CONFIGS["tiny"], 8),
    # 8 sequences x 17 verify rows = 136 rows (three row groups of 48) at a context long enough for key-range
    # splits, head dimension 128: the shape of the batched long-context configuration at reduced width
    "narrow_b8_rows136": (synth.PairConfig("narrow_b8", synth.ModelShape(2, 512, 4, 4, 1024, 4096),
                                           synth.ModelShape(1, 128, 2, 2, 256, 4096), agree=0.8, n_prompt=300,
                                           max_new=24, gamma_max=16), 8),
    # 4 sequences x 13 rows = 52 rows (one group of 64), grouped-query attention
    "gqa_b4_rows52": (synth.PairConfig("gqa_b4", synth.ModelShape(3, 512, 4, 2, 1024, 4096),
                                       synth.ModelShape(2, 256, 4, 2, 512, 4096), agree=0.7, n_prompt=90, max_new=24,
                                       gamma_max=12), 4),
    # 7 sequences x 17 rows = 119 rows (two groups of 64)
    "narrow_b7_rows119": (synth.PairConfig("narrow_b7", synth.ModelShape(2, 256, 2, 2, 512, 4096),
                                           synth.ModelShape(1, 128, 2, 2, 256, 4096), agree=0.8, n_prompt=70,
                                           max_new=24, gamma_max=16), 7),
}


@pytest.fixture(scope="module", params=sorted(WIDE))
def wide(request):
    from paper_2602_01274_b200 import binding as b
    cfg, batch = WIDE[request.param]
    pair_gpu = synth.make_pair(cfg, seed=2, device="cuda:0")
    pair_cpu = {k: ({n: t.cpu() for n, t in v.items()} if isinstance(v, dict) else v.cpu()) for k, v in pair_gpu.items()}
    T, D, B = oracle_models(cfg, pair_cpu)
    max_ctx = cfg.n_prompt + cfg.max_new + cfg.gamma_cap + 2
    ctx = b.Context(b.make_cfg(cfg.target, cfg.draft, batch, max_ctx, cfg.gamma_cap, cfg.block_b, cfg.rho, 0, cfg.succ_bias))
    b.load_pair(ctx, pair_gpu)
    prompts = synth.make_prompts(cfg.target.vocab, batch, cfg.n_prompt, seed=6).numpy()
    yield dict(cfg=cfg, ctx=ctx, T=T, D=D, B=B, prompts=prompts, max_ctx=max_ctx, b=b, batch=batch)
    ctx.close()


def test_wide_verify_logits_against_oracle(wide):
    """One full window per sequence, then ONE verify forward over all sequences' rows: every sequence's logits
    against the oracle's (2e-2), its drafts and alpha_hat too."""
    b, cfg, ctx, batch = wide["b"], wide["cfg"], wide["ctx"], wide["batch"]
    V, gc, bb = cfg.target.vocab, cfg.gamma_cap, cfg.block_b
    ctx.pacer_prefill(wide["prompts"], cfg.max_new, cfg.gamma_max, -1.0)
    for _ in range(gc // bb):
        for _ in range(bb):
            ctx.pacer_draft_step()
        ctx.pacer_preverify()
    ctx.pacer_verify()
    y = ctx.pacer_read_buffer(b.BUF_DRAFTS, np.int32, batch * gc).reshape(batch, gc)
    al = ctx.pacer_read_buffer(b.BUF_ALPHA, np.float32, batch * gc).reshape(batch, gc)
    pl = ctx.pacer_read_buffer(b.BUF_VERIFY_LOGITS, np.float32, batch * (gc + 1) * V).reshape(batch, gc + 1, V)
    for s in range(batch):
        o = orc.Pacer(wide["T"], wide["D"], wide["B"], wide["max_ctx"], b=bb, gamma_cap=gc, t0=-1.0, rho=cfg.rho)
        o.prefill(wide["prompts"][s])
        while o.drafting:
            o.draft_block(); o.preverify()
        o.verify()
        if o.stats()["min_margin_draft"] > 2 * LOGIT_TOL:
            np.testing.assert_array_equal(y[s], o.y(), err_msg=f"sequence {s}")
            assert np.abs(al[s] - o.alpha()).max() < ALPHA_TOL, s
            assert np.abs(pl[s] - o.plogits(gc + 1)).max() < LOGIT_TOL, s


@pytest.mark.parametrize("t0s", [(-1.0,), (0.5, 0.49, 0.505, 0.47, 0.52)])
def test_wide_batch_equals_single_runs(wide, t0s):
    """Every sequence of the batch against the oracle's run of that sequence alone.  A sequence is comparable when
    none of the oracle's decisions lies within tolerance of a tie (with the untrained pre-verification layer the
    block statistic sits near 0.5, so only some sequences and thresholds qualify: several thresholds are tried)."""
    cfg, ctx, batch = wide["cfg"], wide["ctx"], wide["batch"]
    comparable = 0
    for t0 in t0s:
        tok, ns, dl, al, st = ctx.pacer_generate(wide["prompts"], cfg.max_new, cfg.gamma_max, t0)
        ar, _ = ctx.pacer_generate_ar(wide["prompts"], cfg.max_new)
        for s in range(batch):
            o = orc.Pacer(wide["T"], wide["D"], wide["B"], wide["max_ctx"], b=cfg.block_b, gamma_cap=cfg.gamma_cap, t0=t0,
                          rho=cfg.rho)
            out_o, dl_o, al_o, st_o = o.generate(wide["prompts"][s], cfg.max_new)
            safe = st_o["min_margin_target"] > 2 * LOGIT_TOL and st_o["min_margin_draft"] > 2 * LOGIT_TOL and \
                (t0 < 0 or st_o["min_margin_stop"] > ALPHA_TOL)
            if not safe:
                continue
            comparable += 1
            np.testing.assert_array_equal(tok[s], out_o, err_msg=f"sequence {s}")
            np.testing.assert_array_equal(ar[s], out_o, err_msg=f"sequence {s} (autoregressive)")
            assert ns[s] == len(dl_o)
            np.testing.assert_array_equal(dl[s, : ns[s]], dl_o)
            np.testing.assert_array_equal(al[s, : ns[s]], al_o)
    assert comparable >= (batch // 2 if t0s[0] < 0 else 2), comparable
