"""Pins of the oracle's decoding loops: the lossless property (Section 2.2), the
reduction of Algorithm 1 to a fixed window, accounting identities, brute force,
the structural examples the paper prints, and the output law under sampling."""
import dataclasses
import os

import numpy as np
import pytest
import torch

from oracle import pacer_oracle as orc
from paper_2602_01274_b200 import synth
from tests.common import oracle_models, small_pair_config


@pytest.fixture(scope="module")
def tiny():
    cfg = synth.CONFIGS["tiny"]
    pair = synth.make_pair(cfg, seed=0)
    T, D, B = oracle_models(cfg, pair)
    prompt = synth.make_prompts(cfg.target.vocab, 1, cfg.n_prompt, seed=0)[0].numpy()
    ar, margin = orc.generate_ar(T, prompt, cfg.max_new)
    return dict(cfg=cfg, T=T, D=D, B=B, prompt=prompt, ar=ar, ar_margin=margin)


def _pacer(t, t0, **kw):
    cfg = t["cfg"]
    args = dict(b=cfg.block_b, gamma_cap=cfg.gamma_cap, t0=t0, rho=cfg.rho)
    args.update(kw)
    return orc.Pacer(t["T"], t["D"], t["B"], cfg.n_prompt + cfg.max_new + cfg.gamma_cap + 2, **args)


@pytest.mark.parametrize("t0", [-1.0, 0.3, 0.5, 0.7])
def test_greedy_pacer_is_lossless(tiny, t0):
    out, dl, al, st = _pacer(tiny, t0).generate(tiny["prompt"], tiny["cfg"].max_new)
    np.testing.assert_array_equal(out, tiny["ar"])
    b, cap = tiny["cfg"].block_b, tiny["cfg"].gamma_cap
    assert all(g % b == 0 and b <= g <= cap for g in dl)
    assert all(0 <= n <= g for n, g in zip(al, dl))
    total = int((al + 1).sum())
    assert total >= tiny["cfg"].max_new and total - (al[-1] + 1) < tiny["cfg"].max_new
    assert st["n_draft_fwd"] == dl.sum() and st["n_target_fwd"] == len(dl) == st["n_steps"]
    assert st["n_mb_calls"] == (dl // b).sum()


@pytest.mark.parametrize("gamma", [1, 3, 8])
def test_greedy_fixed_window_is_lossless_and_counts_gamma_draft_forwards(tiny, gamma):
    out, dl, al, st = orc.generate_sd(tiny["T"], tiny["D"], tiny["prompt"], tiny["cfg"].max_new, gamma)
    np.testing.assert_array_equal(out, tiny["ar"])
    # Table "num_forward": the draft model is charged exactly gamma forwards per target forward
    assert st["n_draft_fwd"] == gamma * st["n_target_fwd"]


def test_paper_forward_counts_are_exact_multiples():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_structural_examples.txt")
    rows = [l.split() for l in open(path) if l.startswith("numfwd")]
    assert len(rows) == 3
    for r in rows:
        kv = dict(t.split("=") for t in r[2:])
        assert int(kv["draft"]) % int(kv["target"]) == 0
    assert 27423 == 9 * 3047


def test_always_pass_reduces_to_fixed_window(tiny):
    cfg = tiny["cfg"]
    out_p, dl_p, al_p, st_p = _pacer(tiny, -1.0).generate(tiny["prompt"], cfg.max_new)
    out_s, dl_s, al_s, st_s = orc.generate_sd(tiny["T"], tiny["D"], tiny["prompt"], cfg.max_new, cfg.gamma_cap)
    np.testing.assert_array_equal(out_p, out_s)
    np.testing.assert_array_equal(dl_p, dl_s)
    np.testing.assert_array_equal(al_p, al_s)
    assert st_p["n_draft_fwd"] == st_s["n_draft_fwd"] and st_p["n_target_fwd"] == st_s["n_target_fwd"]


def test_threshold_above_one_always_stops_after_one_block(tiny):
    out, dl, al, st = _pacer(tiny, 1.5).generate(tiny["prompt"], tiny["cfg"].max_new)
    assert set(dl.tolist()) == {tiny["cfg"].block_b}
    o2, d2, a2, _ = orc.generate_sd(tiny["T"], tiny["D"], tiny["prompt"], tiny["cfg"].max_new, tiny["cfg"].block_b)
    np.testing.assert_array_equal(al, a2)


def test_accept_lengths_equal_brute_force_common_prefix(tiny):
    """n_s recomputed without the loop: greedy drafts from the true prefix, compared
    token by token with the autoregressive continuation."""
    cfg, T, D = tiny["cfg"], tiny["T"], tiny["D"]
    out, dl, al, _ = _pacer(tiny, 0.5).generate(tiny["prompt"], cfg.max_new)
    assert len(set(dl.tolist())) > 1, "threshold 0.5 should give a varying window on this pair"
    # a longer autoregressive reference, so the last step can be checked too
    ar_long, _ = orc.generate_ar(T, tiny["prompt"], cfg.max_new + cfg.gamma_cap + 1)
    full = np.concatenate([tiny["prompt"], ar_long])
    P = cfg.n_prompt
    for g, n in zip(dl, al):
        c = orc.Cache(D, P + g + 1)
        _, lg = orc.forward(D, c, tokens=full[:P])
        tok = int(lg[-1].argmax())
        drafts = [tok]
        for _ in range(g - 1):
            _, lg = orc.forward(D, c, tokens=[tok])
            tok = int(lg[-1].argmax())
            drafts.append(tok)
        lcp = 0
        while lcp < g and drafts[lcp] == full[P + lcp]:
            lcp += 1
        assert lcp == n
        P += n + 1


def test_threshold_schedule_closed_form_and_equality_stops():
    """t_k = t0 * rho^k inside a step, restarting every step; the test is 'mean <= t'."""
    cfg = small_pair_config(gamma_max=12, b=2)
    pair = synth.make_pair(cfg, seed=1)
    T, D, B = oracle_models(cfg, pair)
    prompt = synth.make_prompts(cfg.target.vocab, 1, 6, seed=1)[0].numpy()
    t0, rho = np.float32(0.4), np.float32(1.25)
    p = orc.Pacer(T, D, B, 64, b=2, gamma_cap=12, t0=float(t0), rho=float(rho))
    p.prefill(prompt)
    t2 = np.float32(np.float32(t0 * rho) * rho)
    # round 0 and 1 pass; round 2: the mean equals t_2 exactly -> must stop ("<=")
    p.set_alpha_override([0.9, 0.9, 0.9, 0.9, float(t2) + 0.25, float(t2) - 0.25])
    ts = []
    while p.drafting:
        ts.append(p.t_k)
        p.draft_block()
        p.preverify()
    assert p.gamma == 6
    np.testing.assert_array_equal(np.array(ts, np.float32), np.array([t0, np.float32(t0 * rho), t2], np.float32))
    np.testing.assert_allclose(ts, [0.4 * 1.25 ** k for k in range(3)], rtol=1e-6)
    p.verify(); p.accept()
    assert p.t_k == t0 and p.gamma == 0 and p.drafting == 1      # restart at the next step
    # just above the threshold the loop goes on
    p.set_alpha_override([float(t0) + 1e-6] * 2 + [0.0, 0.0])
    p.draft_block(); p.preverify()
    assert p.drafting == 1
    p.draft_block(); p.preverify()
    assert p.drafting == 0 and p.gamma == 4


@pytest.mark.parametrize("criterion,alphas,expect_stop", [
    (0, [0.9, 0.2, 0.9, 0.8], False),    # mean 0.7 > 0.5
    (1, [0.9, 0.2, 0.9, 0.8], True),     # any token <= 0.5
    (2, [0.9, 0.2, 0.9, 0.8], False),    # last token 0.8
    (2, [0.9, 0.9, 0.9, 0.4], True),
    (0, [0.9, 0.9, 0.1, 0.0], True),     # mean 0.475
])
def test_halting_criteria(criterion, alphas, expect_stop):
    cfg = small_pair_config(gamma_max=8, b=4)
    pair = synth.make_pair(cfg, seed=2)
    T, D, B = oracle_models(cfg, pair)
    p = orc.Pacer(T, D, B, 64, b=4, gamma_cap=8, t0=0.5, rho=1.0, criterion=criterion)
    p.prefill(synth.make_prompts(cfg.target.vocab, 1, 5, seed=2)[0].numpy())
    p.set_alpha_override(alphas)
    p.draft_block(); p.preverify()
    assert (p.drafting == 0) == expect_stop


def _scripted_pair(chain_T, draft_agree_upto, V=64, seed=5):
    """Models whose next token is dictated by successor tables (bias 50 dwarfs the
    noise logits): the target follows chain_T; the draft agrees on the first
    `draft_agree_upto[i]` links of each listed segment."""
    cfg = small_pair_config(vocab=V)
    cfg = dataclasses.replace(cfg, succ_bias=50.0)
    pair = synth.make_pair(cfg, seed=seed)
    succ_t = torch.arange(V, dtype=torch.int32).roll(-1)        # default: v -> v+1
    succ_d = succ_t.clone()
    for a, b in zip(chain_T[:-1], chain_T[1:]):
        succ_t[a] = b
        succ_d[a] = b
    for tok in draft_agree_upto:                                 # the draft goes astray after `tok`
        succ_d[tok] = 60
    succ_d[60], succ_d[61], succ_d[62] = 61, 62, 63              # and stays astray
    pair["succ_T"], pair["succ_D"] = succ_t, succ_d
    return cfg, oracle_models(cfg, pair)


def test_figure1_scenarios():
    # target text after the prompt's last token 10: 11, 12, ..., ; the draft errs after 17
    chain = list(range(10, 30))
    cfg, (T, D, B) = _scripted_pair(chain, draft_agree_upto=[17])
    prompt = np.array([3, 4, 10], np.int32)
    # (a) block size 3, three rounds, 9 drafts, 7 accepted, one target forward
    p = orc.Pacer(T, D, B, 64, b=3, gamma_cap=12, t0=0.6, rho=1.05)
    p.prefill(prompt)
    p.set_alpha_override([0.9] * 3 + [0.8] * 3 + [0.3] * 3)
    rounds = 0
    while p.drafting:
        p.draft_block(); p.preverify(); rounds += 1
    assert rounds == 3 and p.gamma == 9
    np.testing.assert_array_equal(p.y(), [11, 12, 13, 14, 15, 16, 17, 60, 61])
    p.verify()
    assert p.accept() == 7 and p.last_next == 18
    st = p.stats()
    assert (st["n_target_fwd"], st["n_draft_fwd"], st["n_mb_calls"]) == (1, 9, 3)
    np.testing.assert_array_equal(p.x()[3:], list(range(11, 19)))
    # (b) fixed window 2 needs 3 target and 6 draft forwards for the same 8 tokens
    out, dl, al, st = orc.generate_sd(T, D, prompt, 8, 2)
    np.testing.assert_array_equal(out, list(range(11, 19)))
    assert (st["n_target_fwd"], st["n_draft_fwd"]) == (3, 6)
    # (c) fixed window 9 where the draft errs after two tokens: 9 drafted, 2 accepted
    cfg, (T, D, B) = _scripted_pair(chain, draft_agree_upto=[12])
    out, dl, al, st = orc.generate_sd(T, D, prompt, 3, 9)
    assert dl[0] == 9 and al[0] == 2 and st["n_draft_fwd"] == 9


def test_case_study_scenario():
    """Fixed window 6: six accepted, then six rejected, third forward needed; the
    block-wise loop with b = 3 covers the same text with two target forwards."""
    chain = list(range(10, 30))
    # after 17 (position of the 7th new token) the draft is wrong once, and again after 18
    cfg, (T, D, B) = _scripted_pair(chain, draft_agree_upto=[17, 18])
    prompt = np.array([3, 4, 10], np.int32)
    out, dl, al, st = orc.generate_sd(T, D, prompt, 9, 6)
    assert al.tolist()[:2] == [6, 0] and st["n_target_fwd"] == 3 and st["n_draft_fwd"] == 18
    p = orc.Pacer(T, D, B, 64, b=3, gamma_cap=12, t0=0.6, rho=1.05)
    # step 1: two confident blocks then the cap of the text is near: third block low -> 9 drafts, 7 accepted
    p.prefill(prompt)
    p.set_alpha_override([0.9] * 6 + [0.2] * 3 + [0.1] * 3)
    steps = 0
    while p.P - 3 < 9:
        while p.drafting:
            p.draft_block(); p.preverify()
        p.verify(); p.accept(); steps += 1
    st = p.stats()
    assert steps == 2 and st["n_target_fwd"] == 2 and st["n_draft_fwd"] == 12 < 18
    np.testing.assert_array_equal(p.x()[3:12], out)


def test_all_accepted_step_makes_the_draft_catch_up():
    """After a fully accepted step the draft cache lacks y_gamma: the next step's
    first draft forward takes two rows, still one counted forward, and M_B sees
    the extra row as history."""
    chain = list(range(10, 40))
    cfg, (T, D, B) = _scripted_pair(chain, draft_agree_upto=[])
    p = orc.Pacer(T, D, B, 64, b=2, gamma_cap=4, t0=-1.0, rho=1.0)
    p.prefill(np.array([3, 10], np.int32))
    while p.drafting:
        p.draft_block(); p.preverify()
    p.verify()
    assert p.accept() == 4
    assert p.P == 2 + 5 and p.cache_len(0) == p.P - 1 and p.cache_len(1) == p.P - 2 == p.cache_len(2)
    p.draft_block()
    assert p.n_pend == 3 and p.cache_len(1) == p.P + 1
    p.preverify()
    assert p.cache_len(2) == p.cache_len(1)
    assert p.stats()["n_draft_fwd"] == 6


def test_batch_of_one_state_is_independent_of_history(tiny):
    """Two different thresholds must not leak through shared state: re-running a
    generator object gives the same result as a fresh one."""
    p = _pacer(tiny, 0.5)
    a = p.generate(tiny["prompt"], 24)
    b = p.generate(tiny["prompt"], 24)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])
    np.testing.assert_array_equal(a[2], b[2])


@pytest.mark.parametrize("loop", ["pacer", "sd"])
def test_sampled_output_follows_the_target_distribution(loop):
    """Chi-square of the first two sampled tokens over 20000 seeds against the
    target's exactly enumerated joint distribution (V = 8; sparse cells pooled)."""
    V = 8
    T_s = synth.ModelShape(1, 16, 2, 2, 32, V)
    D_s = synth.ModelShape(1, 16, 2, 1, 24, V)
    wt = synth.make_model(T_s, "target", seed=21, std=0.6)
    wd = synth.make_model(D_s, "draft", seed=22, std=0.6)
    wb = synth.make_model(synth.preverify_shape(D_s), "preverify", seed=23, std=0.6, gamma_cap=4)
    T, D, B = orc.OracleModel(T_s, wt), orc.OracleModel(D_s, wd), orc.OracleModel(synth.preverify_shape(D_s), wb)
    prompt = np.array([1, 5, 2], np.int32)
    # exact joint by teacher forcing
    sm = lambda v: np.exp(v - v.max()) / np.exp(v - v.max()).sum()
    _, lg = orc.forward(T, orc.Cache(T, 8), tokens=prompt)
    p1 = sm(lg[-1])
    joint = np.zeros((V, V))
    for a in range(V):
        _, lg2 = orc.forward(T, orc.Cache(T, 8), tokens=np.append(prompt, a).astype(np.int32))
        joint[a] = p1[a] * sm(lg2[-1])
    N = 20000
    counts = np.zeros((V, V))
    n_acc = 0
    p = orc.Pacer(T, D, B, 16, b=2, gamma_cap=4, t0=0.5, rho=1.05, mode=1)
    for s in range(N):
        if loop == "pacer":
            p.set_seed(7000 + s)
            out, dl, al, _ = p.generate(prompt, 2)
        else:
            out, dl, al, _ = orc.generate_sd(T, D, prompt, 2, 3, mode=1, seed=7000 + s)
        counts[out[0], out[1]] += 1
        n_acc += al[0]
    assert 0.05 * N < n_acc, "the draft should be accepted sometimes"
    exp = (N * joint).ravel()
    cnt = counts.ravel()
    big = exp >= 10.0                    # pool the sparse cells into one
    e = np.append(exp[big], exp[~big].sum())
    c = np.append(cnt[big], cnt[~big].sum())
    assert len(e) >= 8
    from scipy.stats import chi2 as chi2_dist
    chi2 = ((c - e) ** 2 / e).sum()
    assert chi2 < chi2_dist.ppf(0.999, len(e) - 1), (chi2, len(e))


def test_sampled_autoregressive_output_follows_the_target_distribution():
    """Eq. 1 under temperature-1 sampling: the first two tokens the oracle's autoregressive loop draws over 20000
    seeds against the target's exactly enumerated joint distribution (V = 8; sparse cells pooled).  The joint
    comes from the separately pinned forward by teacher forcing, so a wrong position, tag or logit row in the
    sampled loop fails the chi-square."""
    V = 8
    T_s = synth.ModelShape(1, 16, 2, 2, 32, V)
    wt = synth.make_model(T_s, "target", seed=31, std=0.6)
    T = orc.OracleModel(T_s, wt)
    prompt = np.array([4, 0, 6], np.int32)
    sm = lambda v: np.exp(v - v.max()) / np.exp(v - v.max()).sum()
    _, lg = orc.forward(T, orc.Cache(T, 8), tokens=prompt)
    p1 = sm(lg[-1])
    joint = np.zeros((V, V))
    for a in range(V):
        _, lg2 = orc.forward(T, orc.Cache(T, 8), tokens=np.append(prompt, a).astype(np.int32))
        joint[a] = p1[a] * sm(lg2[-1])
    assert joint.max() < 0.6, "the distribution should not be degenerate"
    N = 20000
    counts = np.zeros((V, V))
    for s in range(N):
        out, _ = orc.generate_ar(T, prompt, 2, mode=1, seed=9000 + s)
        counts[out[0], out[1]] += 1
    exp = (N * joint).ravel()
    cnt = counts.ravel()
    big = exp >= 10.0
    e = np.append(exp[big], exp[~big].sum())
    c = np.append(cnt[big], cnt[~big].sum())
    assert len(e) >= 8
    from scipy.stats import chi2 as chi2_dist
    chi2 = ((c - e) ** 2 / e).sum()
    assert chi2 < chi2_dist.ppf(0.999, len(e) - 1), (chi2, len(e))
    # greedy mode of the same loop is the arg-max chain of the same forward
    out_g, _ = orc.generate_ar(T, prompt, 2, mode=0)
    assert out_g[0] == int(np.argmax(p1)) and out_g[1] == int(np.argmax(joint[out_g[0]]))


def test_preverify_inputs_are_hidden_plus_position_embedding_of_the_draft_index():
    """Eq. 7 wiring: row of draft i (1-based within the step, continuing over
    blocks) gets e_i = PosEmb row i-1; a catch-up history row gets none; alpha_hat
    is the second softmax component of the 2-way head.  Rebuilt here from the
    separately pinned layer forward."""
    chain = list(range(10, 40))
    cfg, (T, D, B) = _scripted_pair(chain, draft_agree_upto=[])
    p = orc.Pacer(T, D, B, 64, b=2, gamma_cap=4, t0=-1.0, rho=1.0)
    prompt = np.array([3, 7, 10], np.int32)
    p.prefill(prompt)
    mirror = orc.Cache(B, 64)                       # a second M_B cache fed by this test
    hD, _ = orc.forward(D, orc.Cache(D, 64), tokens=prompt[:-1])
    orc.forward(B, mirror, x_in=hD, want_logits=False)
    posemb = torch.from_numpy(B.keep["posemb"].copy()).view(torch.bfloat16).double().numpy()
    head_b = torch.from_numpy(B.keep["head_b"].copy()).view(torch.bfloat16).double().numpy()
    for step in range(2):
        drafted = 0
        while p.drafting:
            p.draft_block()
            h = p.hpend()
            n_hist = h.shape[0] - 2                 # 1 history row in the step after a full accept
            assert n_hist == (1 if (step == 1 and drafted == 0) else 0)
            xin = h.copy()
            for j in range(2):
                xin[n_hist + j] += posemb[drafted + j]
            hid, _ = orc.forward(B, mirror, x_in=xin, want_logits=False)
            z = hid[n_hist:] @ head_b.T
            expect = np.exp(z[:, 1]) / np.exp(z).sum(1)
            p.preverify()
            np.testing.assert_allclose(p.alpha()[drafted:drafted + 2], expect, atol=1e-12)
            drafted += 2
        p.verify()
        assert p.accept() == 4
        mirror.truncate(p.cache_len(2))


@pytest.mark.parametrize("scope", [1, 2])
def test_restricted_attention_context_of_the_preverification_layer(scope):
    """"Attention context" ablation (Section 5): local block = the drafts of the current block only, local draft =
    the drafts of the current step.  alpha_hat is rebuilt from the separately pinned plain forward run on exactly
    those rows, alone, at positions 0.. (rotary scores depend on position differences only); the second step
    follows a fully accepted one, so its first call carries a catch-up history row that must stay outside."""
    chain = list(range(10, 40))
    cfg, (T, D, B) = _scripted_pair(chain, draft_agree_upto=[])
    p = orc.Pacer(T, D, B, 64, b=2, gamma_cap=4, t0=-1.0, rho=1.0, scope=scope)
    prompt = np.array([3, 7, 10], np.int32)
    p.prefill(prompt)
    posemb = torch.from_numpy(B.keep["posemb"].copy()).view(torch.bfloat16).double().numpy()
    head_b = torch.from_numpy(B.keep["head_b"].copy()).view(torch.bfloat16).double().numpy()
    full = orc.Pacer(T, D, B, 64, b=2, gamma_cap=4, t0=-1.0, rho=1.0, scope=0)
    full.prefill(prompt)
    differs = False
    for step in range(2):
        drafted, step_rows = 0, []
        while p.drafting:
            p.draft_block(); full.draft_block()
            h = p.hpend()
            n_hist = h.shape[0] - 2
            assert n_hist == (1 if (step == 1 and drafted == 0) else 0)
            rows = h[n_hist:].copy()
            for j in range(2):
                rows[j] += posemb[drafted + j]
            step_rows.append(rows)
            ctx_rows = rows if scope == 2 else np.concatenate(step_rows)
            hid, _ = orc.forward(B, orc.Cache(B, 16), x_in=ctx_rows, want_logits=False)
            z = hid[-2:] @ head_b.T
            expect = np.exp(z[:, 1]) / np.exp(z).sum(1)
            p.preverify(); full.preverify()
            np.testing.assert_allclose(p.alpha()[drafted:drafted + 2], expect, atol=1e-9)
            differs |= bool(np.abs(p.alpha()[drafted:drafted + 2] - full.alpha()[drafted:drafted + 2]).max() > 1e-6)
            drafted += 2
        p.verify(); full.verify()
        assert p.accept() == 4 and full.accept() == 4
        assert p.cache_len(2) == full.cache_len(2)
    assert differs, "a restricted context must change alpha_hat"


def test_prescribed_windows_reduce_to_the_fixed_window_and_stay_lossless(tiny):
    """Speculative decoding with a window per step: a constant list is the separately written fixed-window loop,
    any list gives the target's greedy output (Section 2.2), and #draft forwards = the sum of the windows."""
    cfg = tiny["cfg"]
    a = orc.generate_sd(tiny["T"], tiny["D"], tiny["prompt"], cfg.max_new, 4)
    b = orc.generate_sched(tiny["T"], tiny["D"], tiny["prompt"], cfg.max_new, [4])
    for u, v in zip(a[:3], b[:3]):
        np.testing.assert_array_equal(u, v)
    assert a[3]["n_draft_fwd"] == b[3]["n_draft_fwd"]
    windows = [0, 3, 0, 0, 7, 1, 0, 2, 5, 0, 0, 0, 4]
    out, dl, al, st = orc.generate_sched(tiny["T"], tiny["D"], tiny["prompt"], cfg.max_new, windows)
    np.testing.assert_array_equal(out, tiny["ar"])
    want = [windows[min(i, len(windows) - 1)] for i in range(len(dl))]
    np.testing.assert_array_equal(dl, want)
    assert (al <= dl).all() and st["n_draft_fwd"] == int(dl.sum()) and st["n_target_fwd"] == len(dl)
    assert int((al + 1).sum()) >= cfg.max_new > int((al[:-1] + 1).sum())
    # accept lengths are the longest common prefix of the drafts with the target's own continuation (brute force
    # through the fixed-window run started from the same position is covered above; here: a window of 0 is one
    # plain target step)
    assert (al[dl == 0] == 0).all()


def test_optimal_windows_replay_wastes_no_draft(tiny):
    """Section 3.1: take the accepted lengths L_A* of a large-window run as the windows of a second run (the
    optimal draft length gamma*).  The replay meets the same step boundaries, every draft is accepted
    (n_s = gamma_s = L_A*_s), the output is unchanged, and it needs no more target forwards and fewer draft
    forwards than the large-window run."""
    cfg = tiny["cfg"]
    big = orc.generate_sd(tiny["T"], tiny["D"], tiny["prompt"], cfg.max_new, 12)
    out, dl, al, st = orc.generate_sched(tiny["T"], tiny["D"], tiny["prompt"], cfg.max_new, big[2])
    np.testing.assert_array_equal(out, big[0])
    np.testing.assert_array_equal(dl, big[2])
    np.testing.assert_array_equal(al, big[2])
    assert st["n_target_fwd"] == big[3]["n_target_fwd"]
    assert st["n_draft_fwd"] == int(big[2].sum()) < big[3]["n_draft_fwd"]
    assert (big[2] < 12).any() and (big[2] > 0).any()
