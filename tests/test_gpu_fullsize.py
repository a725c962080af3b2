"""GPU parity at the full 7B / 68M, 13B / 68M and 33B / 1.3B sizes, in the launch configuration the benchmark times
(one cooperative launch per forward, one block per SM, 17 or 25 verify rows): all 32 / 40 / 62 layers at width
4096 / 5120 / 7168 (the last with grouped-query attention) and the full LM head, against the fp64 oracle reading
the same bf16 weights.  The prompt is short so that the oracle's prefill stays within seconds; the verify forward
itself is the full one.  One more case runs the 7B pair behind a 520-token prompt (the oracle's prefill then takes a
few minutes): that verify forward has the benchmark's attention shape too, 17 rows against 519 cached keys in 4
key-range splits per head.  Logits within 2e-2; drafts bit-exact where the oracle's margins allow."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import pacer_oracle as orc
from paper_2602_01274_b200 import synth
from tests.common import oracle_models

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2
ALPHA_TOL = 2e-3


@pytest.mark.parametrize("name,n_prompt", [("7b_68m", 4), ("13b_68m", 4), ("33b_1b3", 4), ("7b_68m", 520)])
def test_verify_forward_full_size(name, n_prompt):
    import psutil
    from paper_2602_01274_b200 import binding as b
    need = 2.5 * synth.CONFIGS[name].target.streamed_weight_bytes()      # host copy of the weights + the oracle's buffers
    if psutil.virtual_memory().available < need:
        pytest.skip("not enough host memory for the oracle at this size")
    cfg = dataclasses.replace(synth.CONFIGS[name], n_prompt=n_prompt, max_new=20)
    V, gc, bb = cfg.target.vocab, cfg.gamma_cap, cfg.block_b
    pair_gpu = synth.make_pair(cfg, seed=1, device="cuda:0")
    pair_cpu = {k: ({n: t.cpu() for n, t in v.items()} if isinstance(v, dict) else v.cpu()) for k, v in pair_gpu.items()}
    T, D, B = oracle_models(cfg, pair_cpu)
    max_ctx = cfg.n_prompt + cfg.max_new + gc + 2
    ctx = b.Context(b.make_cfg(cfg.target, cfg.draft, 1, max_ctx, gc, bb, cfg.rho, 0, cfg.succ_bias))
    try:
        b.load_pair(ctx, pair_gpu)
        del pair_gpu
        prompt = synth.make_prompts(V, 1, cfg.n_prompt, seed=3)[0].numpy()
        o = orc.Pacer(T, D, B, max_ctx, b=bb, gamma_cap=gc, t0=-1.0, rho=cfg.rho)
        o.prefill(prompt)
        ctx.pacer_prefill(prompt, cfg.max_new, cfg.gamma_max, -1.0)
        while o.drafting:
            for _ in range(bb):
                ctx.pacer_draft_step()
            o.draft_block()
            ql = ctx.pacer_read_buffer(b.BUF_DRAFT_LOGITS, np.float32, gc * V).reshape(gc, V)[: o.gamma]
            assert np.abs(ql - o.qlogits(o.gamma)).max() < LOGIT_TOL
            y = ctx.pacer_read_buffer(b.BUF_DRAFTS, np.int32, gc)[: o.gamma]
            np.testing.assert_array_equal(y, o.y())
            ctx.pacer_preverify()
            o.preverify()
            al = ctx.pacer_read_buffer(b.BUF_ALPHA, np.float32, gc)[: o.gamma]
            assert np.abs(al - o.alpha()).max() < ALPHA_TOL
        assert o.gamma == gc
        ctx.pacer_verify()
        o.verify()
        pl = ctx.pacer_read_buffer(b.BUF_VERIFY_LOGITS, np.float32, (gc + 1) * V).reshape(gc + 1, V)
        ref = o.plogits(gc + 1)
        err = np.abs(pl - ref).max()
        assert err < LOGIT_TOL, f"verify logits differ by {err}"
        ctx.pacer_accept_rollback()
        n = o.accept()
        st = ctx.pacer_read_state()[0]
        top2 = np.sort(ref, axis=1)[:, -2:]
        if (top2[: n + 1, 1] - top2[: n + 1, 0]).min() > 2 * LOGIT_TOL:
            assert (st["last_n"], st["last_next"], st["P"]) == (n, o.last_next, o.P)
    finally:
        ctx.close()
        torch.cuda.empty_cache()
