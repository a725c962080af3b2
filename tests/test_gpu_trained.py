"""GPU parity with a TRAINED pre-verification layer (the paper's label recipe, trained on the host in the test
session): the CUDA path and the oracle read the same bf16 tensors, and Algorithm 1 must take the same decisions
step by step at the thresholds of the paper's sweep.  With a trained layer alpha_hat sits near 0 or 1, so the stop
decisions clear the tolerance by a wide margin and the adaptive window really varies."""
import numpy as np
import pytest

from oracle import pacer_oracle as orc
from paper_2602_01274_b200 import synth
from tests.common import oracle_models

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2
ALPHA_TOL = 2e-3


def test_trained_layer_same_decisions_as_the_oracle(trained_tiny_preverify):
    from paper_2602_01274_b200 import binding as b
    tensors, report = trained_tiny_preverify
    cfg = synth.CONFIGS["tiny"]
    pair_cpu = synth.make_pair(cfg, seed=0)
    pair_cpu["preverify"] = tensors
    pair_gpu = {k: ({n: t.to("cuda:0") for n, t in v.items()} if isinstance(v, dict) else v.to("cuda:0")) for k, v in pair_cpu.items()}
    T, D, B = oracle_models(cfg, pair_cpu)
    max_ctx = cfg.n_prompt + cfg.max_new + cfg.gamma_cap + 2
    ctx = b.Context(b.make_cfg(cfg.target, cfg.draft, 1, max_ctx, cfg.gamma_cap, cfg.block_b, cfg.rho, 0, cfg.succ_bias))
    try:
        b.load_pair(ctx, pair_gpu)
        compared, varied = 0, 0
        for seed in (77, 78):
            prompt = synth.make_prompts(cfg.target.vocab, 1, cfg.n_prompt, seed=seed)[0].numpy()
            for t0 in (0.3, 0.5, 0.7):
                o = orc.Pacer(T, D, B, max_ctx, b=cfg.block_b, gamma_cap=cfg.gamma_cap, t0=t0, rho=cfg.rho)
                out_o, dl_o, al_o, st_o = o.generate(prompt, cfg.max_new)
                if not (st_o["min_margin_target"] > 2 * LOGIT_TOL and st_o["min_margin_draft"] > 2 * LOGIT_TOL
                        and st_o["min_margin_stop"] > ALPHA_TOL):
                    continue
                tok, ns, dl, al, st = ctx.pacer_generate(prompt, cfg.max_new, cfg.gamma_max, t0)
                np.testing.assert_array_equal(tok[0], out_o)
                assert ns[0] == len(dl_o)
                np.testing.assert_array_equal(dl[0, : ns[0]], dl_o)
                np.testing.assert_array_equal(al[0, : ns[0]], al_o)
                compared += 1
                varied += int(len(set(dl_o.tolist())) > 1)
        assert compared >= 3 and varied >= 2, (compared, varied)
    finally:
        ctx.close()
