"""GPU parity of speculative decoding with prescribed windows (pacer_generate_sched) and of the optimal-window replay
of Section 3.1: the windows of a second run are the accepted lengths L_A* of a large-window run, every draft is then
accepted and the output is unchanged.  Against the CPU oracle's separately written loop on the same seeded inputs:
tokens and per-step (window, accepted) bit-exact where the oracle's deciding margins exceed the tolerance.  Also the
error path of the device status word, exercised from the host (no kernel is made to fail)."""
import numpy as np
import pytest

from oracle import pacer_oracle as orc
from paper_2602_01274_b200 import synth
from tests.common import oracle_models

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2


@pytest.fixture(scope="module")
def tiny2():
    from paper_2602_01274_b200 import binding as b
    cfg = synth.CONFIGS["tiny"]
    pair_gpu = synth.make_pair(cfg, seed=0, device="cuda:0")
    pair_cpu = {k: ({n: t.cpu() for n, t in v.items()} if isinstance(v, dict) else v.cpu()) for k, v in pair_gpu.items()}
    T, D, B = oracle_models(cfg, pair_cpu)
    max_ctx = cfg.n_prompt + cfg.max_new + cfg.gamma_cap + 2
    ctx = b.Context(b.make_cfg(cfg.target, cfg.draft, 2, max_ctx, cfg.gamma_cap, cfg.block_b, cfg.rho, 0, cfg.succ_bias))
    b.load_pair(ctx, pair_gpu)
    prompts = synth.make_prompts(cfg.target.vocab, 2, cfg.n_prompt, seed=0).numpy()
    yield dict(cfg=cfg, ctx=ctx, T=T, D=D, prompts=prompts, max_ctx=max_ctx, b=b)
    ctx.close()


def _safe(st):
    return st["min_margin_target"] > 2 * LOGIT_TOL and st["min_margin_draft"] > 2 * LOGIT_TOL


@pytest.mark.parametrize("windows", [[3], [0, 3, 0, 0, 7, 1, 0, 2, 5, 0, 0, 0, 4], [8, 0, 0, 0, 0, 2], [0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 1]])
def test_prescribed_windows_match_oracle(tiny2, windows):
    cfg, ctx = tiny2["cfg"], tiny2["ctx"]
    prompt = tiny2["prompts"][0]
    out_o, dl_o, al_o, st_o = orc.generate_sched(tiny2["T"], tiny2["D"], prompt, cfg.max_new, windows, max_ctx=tiny2["max_ctx"])
    assert _safe(st_o)
    tok, ns, dl, al, st = ctx.pacer_generate_sched(prompt, cfg.max_new, windows)
    np.testing.assert_array_equal(tok[0], out_o)
    assert ns[0] == len(dl_o)
    np.testing.assert_array_equal(dl[0, : ns[0]], dl_o)
    np.testing.assert_array_equal(al[0, : ns[0]], al_o)
    assert st["n_draft_fwd"] == st_o["n_draft_fwd"] and st["n_target_fwd"] == st_o["n_target_fwd"] and st["n_mb_calls"] == 0


def test_draft_backlog_limit_turns_a_zero_window_into_one(tiny2):
    """Windows of 0 forever: the draft model falls one row further behind per step, and a draft forward holds 16
    rows per sequence here, so every 16th step or so must draft one token (the documented limit of the entry
    point).  The output is the target's own greedy text all the same."""
    cfg, ctx = tiny2["cfg"], tiny2["ctx"]
    prompt = tiny2["prompts"][0]
    tok, ns, dl, al, st = ctx.pacer_generate_sched(prompt, cfg.max_new, [0])
    ar, _ = ctx.pacer_generate_ar(prompt, cfg.max_new)
    np.testing.assert_array_equal(tok[0], ar[0])
    w = dl[0, : ns[0]]
    assert set(w.tolist()) == {0, 1} and int(w.sum()) >= 2
    runs = np.diff(np.flatnonzero(np.concatenate([[1], w, [1]])))
    assert runs.max() - 1 <= 15
    assert (w[:15] == 0).all() and w[15] == 1


def test_optimal_window_replay(tiny2):
    """gamma* of Section 3.1 on the device: L_A* from a run with the largest window, replayed as the windows."""
    cfg, ctx = tiny2["cfg"], tiny2["ctx"]
    prompt = tiny2["prompts"][0]
    tok_big, ns_big, dl_big, al_big, st_big = ctx.pacer_generate(prompt, cfg.max_new, cfg.gamma_cap, -1.0)
    la = al_big[0, : ns_big[0]]
    tok, ns, dl, al, st = ctx.pacer_generate_sched(prompt, cfg.max_new, la)
    np.testing.assert_array_equal(tok[0], tok_big[0])
    assert ns[0] == ns_big[0]
    np.testing.assert_array_equal(dl[0, : ns[0]], la)
    np.testing.assert_array_equal(al[0, : ns[0]], la)
    assert st["n_draft_fwd"] == int(la.sum()) < st_big["n_draft_fwd"] and st["n_target_fwd"] == st_big["n_target_fwd"]
    # and the oracle's replay of its own large-window run gives the same schedule and tokens
    big_o = orc.generate_sd(tiny2["T"], tiny2["D"], prompt, cfg.max_new, cfg.gamma_cap)
    assert _safe(big_o[3])
    np.testing.assert_array_equal(big_o[2], la)
    np.testing.assert_array_equal(big_o[0], tok[0])


def test_prescribed_windows_per_sequence_in_a_batch(tiny2):
    cfg, ctx = tiny2["cfg"], tiny2["ctx"]
    windows = np.array([[2, 0, 5, 1, 0, 0, 3, 8], [0, 0, 4, 4, 1, 6, 0, 2]], np.int32)
    tok, ns, dl, al, _ = ctx.pacer_generate_sched(tiny2["prompts"], cfg.max_new, windows)
    for s in range(2):
        out_o, dl_o, al_o, st_o = orc.generate_sched(tiny2["T"], tiny2["D"], tiny2["prompts"][s], cfg.max_new, windows[s],
                                                     max_ctx=tiny2["max_ctx"])
        assert _safe(st_o)
        np.testing.assert_array_equal(tok[s], out_o)
        assert ns[s] == len(dl_o)
        np.testing.assert_array_equal(dl[s, : ns[s]], dl_o)
        np.testing.assert_array_equal(al[s, : ns[s]], al_o)


def test_prescribed_windows_bad_arguments(tiny2):
    b, cfg, ctx = tiny2["b"], tiny2["cfg"], tiny2["ctx"]
    with pytest.raises(b.PacerError):
        ctx.pacer_generate_sched(tiny2["prompts"][0], cfg.max_new, [cfg.gamma_cap + 1])
    with pytest.raises(b.PacerError):
        ctx.pacer_generate_sched(tiny2["prompts"][0], cfg.max_new, [-1])


def test_device_status_word_reaches_the_host_as_an_error(tiny2):
    """The word a kernel's bounded wait leaves behind when it gives up is written from the host here; every
    synchronising entry point must then report PACER_EDEVICE with the decoded record, and the next run clears it."""
    b, cfg, ctx = tiny2["b"], tiny2["cfg"], tiny2["ctx"]
    prompt = tiny2["prompts"][0]
    ctx.pacer_generate(prompt, 8, cfg.gamma_max, -1.0)
    ctx.pacer_debug_set_device_status(9, 17, 9, 1234)
    for call in (lambda: ctx.pacer_read_state(), lambda: ctx.pacer_read_buffer(b.BUF_TOKENS, np.int32, 4)):
        with pytest.raises(b.PacerError) as e:
            call()
        assert "device-side anomaly" in str(e.value) and "wait code 9" in str(e.value) and "block 17" in str(e.value) \
            and "detail 1234" in str(e.value)
    tok, *_ = ctx.pacer_generate(prompt, 8, cfg.gamma_max, -1.0)      # a new run resets the word
    assert ctx.pacer_read_state()[0]["finished"] == 1
    ref, _ = ctx.pacer_generate_ar(prompt, 8)
    np.testing.assert_array_equal(tok[0], ref[0])
