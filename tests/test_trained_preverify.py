"""The pre-verification layer trained with the paper's recipe (Section 3.3: the target's responses, drafts from every
prefix, labels 1..1 0..0 up to the first mismatch, cross-entropy, AdamW) on the tiny synthetic pair.  The training
job is plain PyTorch outside the decoding path; here its result is loaded into the CPU oracle: the scores the
oracle's own M_B forward gives during decoding must separate accepted from rejected drafts, and Algorithm 1 driven by
them must waste fewer draft forwards than any fixed window that accepts as many tokens per step."""
import numpy as np
import pytest

from oracle import pacer_oracle as orc
from paper_2602_01274_b200 import synth, train_preverify
from tests.common import oracle_models


@pytest.fixture(scope="module")
def tiny_trained(trained_tiny_preverify):
    tensors, report = trained_tiny_preverify
    cfg = synth.CONFIGS["tiny"]
    pair = synth.make_pair(cfg, seed=0)
    pair["preverify"] = tensors
    T, D, B = oracle_models(cfg, pair)
    prompts = synth.make_prompts(cfg.target.vocab, 4, cfg.n_prompt, seed=77).numpy()
    return dict(cfg=cfg, T=T, D=D, B=B, prompts=prompts, report=report)


def test_training_report(tiny_trained):
    rep = tiny_trained["report"]
    assert rep["held_out_auc"] > 0.95, rep
    assert rep["mean_alpha_accepted"] > 0.8 and rep["mean_alpha_rejected"] < 0.2, rep


def test_oracle_scores_with_trained_layer_separate_accepted_from_rejected_drafts(tiny_trained):
    """Through the oracle's own M_B forward and cache handling (not the training script's): full windows, then
    alpha_hat of every draft against what the acceptance step decided."""
    import torch
    t = tiny_trained
    cfg = t["cfg"]
    scores, labels = [], []
    for prompt in t["prompts"]:
        o = orc.Pacer(t["T"], t["D"], t["B"], cfg.n_prompt + 64 + cfg.gamma_cap + 2, b=cfg.block_b, gamma_cap=cfg.gamma_cap,
                      t0=-1.0, rho=cfg.rho)
        o.prefill(prompt)
        while o.P - cfg.n_prompt < 48:
            while o.drafting:
                o.draft_block(); o.preverify()
            alpha = o.alpha().copy()
            o.verify()
            n = o.accept()
            scores.append(alpha)
            labels.append((np.arange(len(alpha)) < n).astype(np.int64))
    a = train_preverify.auc(torch.from_numpy(np.concatenate(scores)), torch.from_numpy(np.concatenate(labels)))
    assert a > 0.9, a


def test_trained_pacer_is_lossless_and_wastes_fewer_drafts(tiny_trained):
    t = tiny_trained
    cfg = t["cfg"]
    max_ctx = cfg.n_prompt + cfg.max_new + cfg.gamma_cap + 2
    for prompt in t["prompts"][:2]:
        ar, _ = orc.generate_ar(t["T"], prompt, cfg.max_new)
        o = orc.Pacer(t["T"], t["D"], t["B"], max_ctx, b=cfg.block_b, gamma_cap=cfg.gamma_cap, t0=0.5, rho=cfg.rho)
        out, dl, al, st = o.generate(prompt, cfg.max_new)
        np.testing.assert_array_equal(out, ar)                         # Section 2.2: the output is the target's own
        assert len(set(dl.tolist())) > 1, "the window should vary from step to step"
        waste = (dl - al).sum() / dl.sum()
        for g in (4, 8):
            _, dl_f, al_f, _ = orc.generate_sd(t["T"], t["D"], prompt, cfg.max_new, g)
            if al_f.mean() >= al.mean() - 0.25:                        # a fixed window that accepts about as much per step
                assert waste < (dl_f - al_f).sum() / dl_f.sum()
