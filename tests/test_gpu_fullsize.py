"""GPU parity at the full 7B / 68M, 13B / 68M and 33B / 1.3B sizes, in the launch configuration the benchmark times
(one cooperative launch per forward, one block per SM, 17 or 25 verify rows): all 32 / 40 / 62 layers at width
4096 / 5120 / 7168 (the last with grouped-query attention) and the full LM head, against the fp64 oracle reading
the same bf16 weights.  The prompt is short so that the oracle's prefill stays within seconds; the verify forward
itself is the full one.  One more case runs the 7B pair behind a 280-token prompt (the oracle's prefill then takes a
few minutes): that verify forward has the benchmark's attention shape too, 17 rows against 279 cached keys in 4
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


@pytest.mark.parametrize("name,n_prompt", [("7b_68m", 4), ("13b_68m", 4), ("33b_1b3", 4), ("qwen_32b_1b5", 4), ("7b_68m", 280)])
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


def test_batched_verify_forward_full_size():
    """The batched configuration at full 7B / 68M width: 8 sequences x 17 rows = 136 rows in ONE verify forward
    (three row groups, each with its own accumulator), every sequence against the oracle's run of that sequence."""
    import psutil
    from paper_2602_01274_b200 import binding as b
    base = synth.CONFIGS["7b_68m_long_b8"]
    if psutil.virtual_memory().available < 2.5 * base.target.streamed_weight_bytes():
        pytest.skip("not enough host memory for the oracle at this size")
    cfg = dataclasses.replace(base, n_prompt=6, max_new=20)
    V, gc, bb, batch = cfg.target.vocab, cfg.gamma_cap, cfg.block_b, cfg.batch
    pair_gpu = synth.make_pair(cfg, seed=1, device="cuda:0")
    pair_cpu = {k: ({n: t.cpu() for n, t in v.items()} if isinstance(v, dict) else v.cpu()) for k, v in pair_gpu.items()}
    T, D, B = oracle_models(cfg, pair_cpu)
    max_ctx = cfg.n_prompt + cfg.max_new + gc + 2
    ctx = b.Context(b.make_cfg(cfg.target, cfg.draft, batch, max_ctx, gc, bb, cfg.rho, 0, cfg.succ_bias))
    try:
        b.load_pair(ctx, pair_gpu)
        del pair_gpu
        prompts = synth.make_prompts(V, batch, cfg.n_prompt, seed=3).numpy()
        ctx.pacer_prefill(prompts, cfg.max_new, cfg.gamma_max, -1.0)
        for _ in range(gc // bb):
            for _ in range(bb):
                ctx.pacer_draft_step()
            ctx.pacer_preverify()
        ctx.pacer_verify()
        y = ctx.pacer_read_buffer(b.BUF_DRAFTS, np.int32, batch * gc).reshape(batch, gc)
        al = ctx.pacer_read_buffer(b.BUF_ALPHA, np.float32, batch * gc).reshape(batch, gc)
        pl = ctx.pacer_read_buffer(b.BUF_VERIFY_LOGITS, np.float32, batch * (gc + 1) * V).reshape(batch, gc + 1, V)
        ctx.pacer_accept_rollback()
        st = ctx.pacer_read_state(batch)
        checked = 0
        for s in (0, 3, 7):                       # three of the eight sequences keep the oracle within a minute
            o = orc.Pacer(T, D, B, max_ctx, b=bb, gamma_cap=gc, t0=-1.0, rho=cfg.rho)
            o.prefill(prompts[s])
            while o.drafting:
                o.draft_block(); o.preverify()
            o.verify()
            if o.stats()["min_margin_draft"] <= 2 * LOGIT_TOL:
                continue
            np.testing.assert_array_equal(y[s], o.y(), err_msg=f"sequence {s}")
            assert np.abs(al[s] - o.alpha()).max() < ALPHA_TOL, s
            ref = o.plogits(gc + 1)
            err = np.abs(pl[s] - ref).max()
            assert err < LOGIT_TOL, f"sequence {s}: verify logits differ by {err}"
            n = o.accept()
            top2 = np.sort(ref, axis=1)[:, -2:]
            if (top2[: n + 1, 1] - top2[: n + 1, 0]).min() > 2 * LOGIT_TOL:
                assert (st[s]["last_n"], st[s]["last_next"], st[s]["P"]) == (n, o.last_next, o.P)
            checked += 1
        assert checked >= 2
    finally:
        ctx.close()
        torch.cuda.empty_cache()
