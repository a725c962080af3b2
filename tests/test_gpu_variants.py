"""GPU parity of the method's switches (the ablations of Section 4.3 and Appendix B are parameters of the same
kernels): halting criterion mean / any token / last token, the draft position embedding switched off, other block
sizes b and growth factors rho, and the attention context of the pre-verification layer (full / local draft / local
block).  Whole runs of Algorithm 1 on the tiny pair, compared with the oracle token for
token and step for step; the comparison is asserted where the oracle's deciding margins exceed the tolerances."""
import numpy as np
import pytest

from oracle import pacer_oracle as orc
from paper_2602_01274_b200 import synth
from tests.common import oracle_models

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2
ALPHA_TOL = 2e-3

# (criterion, use_posemb, block b, rho, attention context of M_B: 0 full, 1 local draft, 2 local block)
VARIANTS = [(1, 1, 4, 1.05, 0), (2, 1, 4, 1.05, 0), (0, 0, 4, 1.05, 0), (0, 1, 2, 1.05, 0), (0, 1, 1, 1.05, 0),
            (0, 1, 4, 1.2, 0), (1, 0, 2, 1.0, 0), (0, 1, 4, 1.05, 1), (0, 1, 4, 1.05, 2), (0, 1, 2, 1.05, 1), (0, 1, 2, 1.0, 2)]


@pytest.fixture(scope="module")
def pair():
    cfg = synth.CONFIGS["tiny"]
    pair_gpu = synth.make_pair(cfg, seed=0, device="cuda:0")
    pair_cpu = {k: ({n: t.cpu() for n, t in v.items()} if isinstance(v, dict) else v.cpu()) for k, v in pair_gpu.items()}
    T, D, B = oracle_models(cfg, pair_cpu)
    prompt = synth.make_prompts(cfg.target.vocab, 1, cfg.n_prompt, seed=0)[0].numpy()
    return dict(cfg=cfg, pair_gpu=pair_gpu, T=T, D=D, B=B, prompt=prompt)


@pytest.mark.parametrize("criterion,use_posemb,bb,rho,scope", VARIANTS)
def test_variant_matches_oracle(pair, criterion, use_posemb, bb, rho, scope):
    from paper_2602_01274_b200 import binding as b
    cfg = pair["cfg"]
    gamma_cap = cfg.gamma_max // bb * bb
    max_ctx = cfg.n_prompt + cfg.max_new + gamma_cap + 2
    ctx = b.Context(b.make_cfg(cfg.target, cfg.draft, 1, max_ctx, gamma_cap, bb, rho, criterion, cfg.succ_bias, use_posemb, scope))
    try:
        b.load_pair(ctx, pair["pair_gpu"])
        compared = 0
        for t0 in (0.49, 0.505, 0.47, 0.52):
            o = orc.Pacer(pair["T"], pair["D"], pair["B"], max_ctx, b=bb, gamma_cap=gamma_cap, t0=t0, rho=rho,
                          criterion=criterion, use_posemb=use_posemb, scope=scope)
            out_o, dl_o, al_o, st_o = o.generate(pair["prompt"], cfg.max_new)
            if not (st_o["min_margin_target"] > 2 * LOGIT_TOL and st_o["min_margin_draft"] > 2 * LOGIT_TOL
                    and st_o["min_margin_stop"] > ALPHA_TOL):
                continue                      # a decision of this run sits within tolerance of a tie: not comparable
            tok, ns, dl, al, st = ctx.pacer_generate(pair["prompt"], cfg.max_new, cfg.gamma_max, t0)
            np.testing.assert_array_equal(tok[0], out_o)
            assert ns[0] == len(dl_o)
            np.testing.assert_array_equal(dl[0, : ns[0]], dl_o)
            np.testing.assert_array_equal(al[0, : ns[0]], al_o)
            assert st["n_draft_fwd"] == st_o["n_draft_fwd"] and st["n_mb_calls"] == st_o["n_mb_calls"]
            compared += 1
        assert compared >= 1, "no threshold gave a run with safe margins"
    finally:
        ctx.close()
