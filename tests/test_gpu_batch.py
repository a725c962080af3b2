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
