"""Pins of the oracle's decoder forward against things other than itself:
a formulation built from torch library routines (complex-number rotary, library
softmax attention, matmul), closed forms and special cases."""
import dataclasses
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import pacer_oracle as orc
from paper_2602_01274_b200 import synth

torch.set_num_threads(4)


def _torch_decoder(shape, w, tokens, x_in=None, succ=None, succ_bias=0.0):
    """Whole-sequence causal decoder from library routines, float64.
    Rotary embedding as multiplication of complex pairs (x_i + i*x_{i+hd/2})."""
    w = {k: v.double() for k, v in w.items()}
    d, H, Hkv, hd = shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim
    x = w["embed"][torch.as_tensor(tokens, dtype=torch.long)] if x_in is None else torch.as_tensor(x_in).double()
    n = x.shape[0]
    pos = torch.arange(n, dtype=torch.float64)
    inv = shape.rope_theta ** (-torch.arange(0, hd // 2, dtype=torch.float64) * 2.0 / hd)
    rot = torch.polar(torch.ones(n, hd // 2, dtype=torch.float64), pos[:, None] * inv[None, :])  # [n][hd/2]

    def rope(t):  # t [n][heads][hd]
        c = torch.complex(t[..., : hd // 2], t[..., hd // 2:]) * rot[:, None, :]
        return torch.cat([c.real, c.imag], dim=-1)

    def rms(t, g):
        return t * torch.rsqrt(t.pow(2).mean(-1, keepdim=True) + shape.rms_eps) * g

    for l in range(shape.n_layers):
        a = rms(x, w["norm1"][l])
        qkv = a @ w["wqkv"][l].T
        q = rope(qkv[:, : H * hd].view(n, H, hd))
        k = rope(qkv[:, H * hd: (H + Hkv) * hd].view(n, Hkv, hd))
        v = qkv[:, (H + Hkv) * hd:].view(n, Hkv, hd)
        k = k.repeat_interleave(H // Hkv, dim=1)
        v = v.repeat_interleave(H // Hkv, dim=1)
        att = F.scaled_dot_product_attention(q.transpose(0, 1), k.transpose(0, 1), v.transpose(0, 1), is_causal=True)
        x = x + att.transpose(0, 1).reshape(n, H * hd) @ w["wo"][l].T
        m = rms(x, w["norm2"][l])
        x = x + (F.silu(m @ w["wgate"][l].T) * (m @ w["wup"][l].T)) @ w["wdown"][l].T
    hid = rms(x, w["normf"])
    logits = None
    if "head" in w:
        logits = hid @ w["head"].T
        if succ is not None:
            for r in range(n):
                logits[r, succ[tokens[r]]] += succ_bias
    return hid.numpy(), None if logits is None else logits.numpy()


def _random_model(shape, which, seed, std=0.3, gains=True, gamma_cap=4):
    w = synth.make_model(shape, which, seed=seed, std=std, gamma_cap=gamma_cap)
    if gains:  # non-unit gains so that a dropped or misplaced gain shows
        for k in ("norm1", "norm2", "normf"):
            w[k] = (1.0 + synth.normal_bf16(seed + 7, 50 + len(k) + ord(k[-1]), w[k].shape, std=0.3)).to(torch.bfloat16)
    return w


SHAPES = [
    synth.ModelShape(2, 32, 4, 4, 48, 40),     # MHA
    synth.ModelShape(3, 48, 6, 2, 64, 33),     # grouped KV heads, odd vocabulary
]


@pytest.mark.parametrize("shape", SHAPES)
def test_forward_matches_library_formulation(shape):
    w = _random_model(shape, "target", seed=3)
    succ, _ = synth.make_succ_tables(shape.vocab, 0.5, seed=3)
    tokens = synth.make_prompts(shape.vocab, 1, 11, seed=5)[0].numpy()
    m = orc.OracleModel(shape, w, succ, 2.5)
    c = orc.Cache(m, 16)
    hid, lg = orc.forward(m, c, tokens=tokens)
    hid_t, lg_t = _torch_decoder(shape, w, tokens, succ=succ.numpy(), succ_bias=2.5)
    assert c.len == 11
    np.testing.assert_allclose(hid, hid_t, rtol=0, atol=1e-9)
    np.testing.assert_allclose(lg, lg_t, rtol=0, atol=1e-9)


def test_parallel_forward_equals_sequential_cached_forwards():
    """Eq. 2 against Eq. 1: m rows at once == m cached single-row steps, and a
    split into chunks in between, to rounding order (here: exactly)."""
    shape = SHAPES[1]
    w = _random_model(shape, "target", seed=1)
    tokens = synth.make_prompts(shape.vocab, 1, 9, seed=2)[0].numpy()
    m = orc.OracleModel(shape, w)
    c1, c2, c3 = orc.Cache(m, 12), orc.Cache(m, 12), orc.Cache(m, 12)
    h_all, l_all = orc.forward(m, c1, tokens=tokens)
    rows = [orc.forward(m, c2, tokens=tokens[i:i + 1]) for i in range(9)]
    np.testing.assert_array_equal(h_all, np.concatenate([r[0] for r in rows]))
    np.testing.assert_array_equal(l_all, np.concatenate([r[1] for r in rows]))
    a = orc.forward(m, c3, tokens=tokens[:4])
    b = orc.forward(m, c3, tokens=tokens[4:])
    np.testing.assert_array_equal(l_all, np.concatenate([a[1], b[1]]))
    k1, v1 = c1.kv()
    k2, v2 = c2.kv()
    np.testing.assert_array_equal(k1, k2)
    np.testing.assert_array_equal(v1, v2)


def test_cache_truncate_then_rewrite_equals_fresh_run():
    """Rolling the cache back and writing other rows leaves no trace of the dropped rows."""
    shape = SHAPES[0]
    w = _random_model(shape, "target", seed=4)
    m = orc.OracleModel(shape, w)
    t1 = np.array([1, 2, 3, 4, 5, 6], np.int32)
    t2 = np.array([1, 2, 3, 9, 8], np.int32)
    c = orc.Cache(m, 8)
    orc.forward(m, c, tokens=t1)
    c.truncate(3)
    _, l_roll = orc.forward(m, c, tokens=t2[3:])
    _, l_fresh = orc.forward(m, orc.Cache(m, 8), tokens=t2)
    np.testing.assert_array_equal(l_roll, l_fresh[3:])


def test_zero_layers_reduce_to_norm_and_head():
    """With every layer matrix zero the residual stream is the embedding, so
    hidden = RMSNorm(E[tok]) * g and logits = head @ hidden (closed form)."""
    shape = SHAPES[0]
    w = _random_model(shape, "target", seed=6)
    for k in ("wqkv", "wo", "wgate", "wup", "wdown"):
        w[k] = torch.zeros_like(w[k])
    m = orc.OracleModel(shape, w)
    tokens = np.array([5, 17, 3], np.int32)
    hid, lg = orc.forward(m, orc.Cache(m, 4), tokens=tokens)
    e = w["embed"].double()[tokens.astype(np.int64)]
    ref = e / torch.sqrt((e * e).mean(-1, keepdim=True) + shape.rms_eps) * w["normf"].double()
    np.testing.assert_allclose(hid, ref.numpy(), atol=1e-12)
    np.testing.assert_allclose(lg, (ref @ w["head"].double().T).numpy(), atol=1e-12)


def test_single_row_attention_is_value_passthrough():
    """One token at position 0: softmax over one key is 1 and the rotary angle is
    0, so the layer is x + Wo Wv norm(x) + MLP: closed form with plain matmuls."""
    shape = dataclasses.replace(SHAPES[1], n_layers=1)
    w = _random_model(shape, "target", seed=8)
    m = orc.OracleModel(shape, w)
    hid, _ = orc.forward(m, orc.Cache(m, 2), tokens=np.array([7], np.int32))
    W = {k: v.double() for k, v in w.items()}
    H, Hkv, hd = shape.n_heads, shape.n_kv_heads, shape.head_dim
    rms = lambda t, g: t / torch.sqrt((t * t).mean() + shape.rms_eps) * g
    x = W["embed"][7]
    v = (W["wqkv"][0] @ rms(x, W["norm1"][0]))[(H + Hkv) * hd:].view(Hkv, hd)
    att = v.repeat_interleave(H // Hkv, dim=0).reshape(-1)
    x = x + W["wo"][0] @ att
    mm = rms(x, W["norm2"][0])
    x = x + W["wdown"][0] @ (F.silu(W["wgate"][0] @ mm) * (W["wup"][0] @ mm))
    np.testing.assert_allclose(hid[0], rms(x, W["normf"]).numpy(), atol=1e-10)


def test_uniform_attention_when_queries_vanish():
    """Zero query weights give equal scores, so each row's attention output is the
    running mean of the values of rows 0..j: pins the causal extent (keys 0..pos,
    the row itself included)."""
    shape = dataclasses.replace(SHAPES[0], n_layers=1)
    w = _random_model(shape, "target", seed=9)
    H, hd = shape.n_heads, shape.head_dim
    w["wqkv"][0, : H * hd] = 0
    for k in ("wgate", "wup", "wdown"):
        w[k] = torch.zeros_like(w[k])
    w["wo"][0] = torch.eye(shape.d_model, dtype=torch.bfloat16)
    w["normf"] = torch.ones_like(w["normf"])
    m = orc.OracleModel(shape, w)
    tokens = np.array([1, 2, 3, 4, 5], np.int32)
    # hidden = RMSNorm(x + cumulative mean of v): recover the pre-norm vector up to scale
    hid, _ = orc.forward(m, orc.Cache(m, 8), tokens=tokens)
    W = {k: v.double() for k, v in w.items()}
    x = W["embed"][tokens.astype(np.int64)]
    a = x / torch.sqrt((x * x).mean(-1, keepdim=True) + shape.rms_eps) * W["norm1"][0]
    v = a @ W["wqkv"][0][2 * H * hd:].T
    run = torch.cumsum(v, 0) / torch.arange(1, 6, dtype=torch.float64)[:, None]
    y = x + run
    ref = y / torch.sqrt((y * y).mean(-1, keepdim=True) + shape.rms_eps)
    np.testing.assert_allclose(hid, ref.numpy(), atol=1e-10)


def test_bf16_weights_equal_their_fp32_expansion():
    shape = SHAPES[0]
    w = _random_model(shape, "target", seed=10)
    tokens = np.array([3, 1, 4, 1, 5], np.int32)
    m16 = orc.OracleModel(shape, w)
    m32 = orc.OracleModel(shape, {k: v.float() for k, v in w.items()})
    a = orc.forward(m16, orc.Cache(m16, 8), tokens=tokens)
    b = orc.forward(m32, orc.Cache(m32, 8), tokens=tokens)
    np.testing.assert_array_equal(a[1], b[1])


def test_preverify_layer_without_embedding_is_a_plain_layer_and_blockwise_equals_full():
    """M_B on a hidden-state sequence: feeding it block by block against its own
    cache equals one causal pass over the whole sequence (library formulation)."""
    shape = synth.ModelShape(1, 32, 4, 4, 48, 40)
    w = _random_model(shape, "preverify", seed=11)
    m = orc.OracleModel(shape, w)
    xin = synth.normal_bf16(12, 77, (10, 32), std=1.0).double().numpy()
    c = orc.Cache(m, 12)
    parts = [orc.forward(m, c, x_in=xin[s:e], want_logits=False)[0] for s, e in ((0, 3), (3, 7), (7, 10))]
    hid_t, _ = _torch_decoder(shape, w, None, x_in=xin)
    np.testing.assert_allclose(np.concatenate(parts), hid_t, atol=1e-9)


def test_linear_helper_is_a_matmul():
    w = synth.normal_bf16(1, 5, (37, 24), std=1.0)
    x = np.random.default_rng(0).normal(size=(3, 24))
    np.testing.assert_allclose(orc.linear(w, x), x @ w.double().numpy().T, atol=1e-12)


def test_restricted_context_equals_the_suffix_run_alone_at_position_zero():
    """The "attention context" variants of the pre-verification layer restrict a row to the cache positions from
    key_start on.  Rotary scores depend on position differences only, so rows that start at key_start and see
    nothing before it must come out exactly as the same rows run alone, at positions 0.., on an empty cache
    (the plain forward, pinned above).  A dropped lower bound, an off-by-one in it, or a bound applied to the
    values but not the scores all break the equality."""
    shape = synth.ModelShape(1, 32, 4, 2, 48, 40)
    w = _random_model(shape, "preverify", seed=11)
    m = orc.OracleModel(shape, w)
    rng = np.random.default_rng(3)
    hist, blk = rng.standard_normal((5, 32)), rng.standard_normal((4, 32))
    full = orc.Cache(m, 16)
    orc.forward(m, full, x_in=hist, want_logits=False)
    got, _ = orc.forward(m, full, x_in=blk, want_logits=False, key_start=5)
    alone, _ = orc.forward(m, orc.Cache(m, 16), x_in=blk, want_logits=False)
    np.testing.assert_allclose(got, alone, atol=1e-9)
    # with the bound one position earlier the last history row is visible and the result must differ
    full.truncate(5)
    other, _ = orc.forward(m, full, x_in=blk, want_logits=False, key_start=4)
    assert np.abs(other - alone).max() > 1e-4
    # key_start = 0 is the ordinary forward
    full.truncate(5)
    a, _ = orc.forward(m, full, x_in=blk, want_logits=False, key_start=0)
    full.truncate(5)
    b, _ = orc.forward(m, full, x_in=blk, want_logits=False)
    np.testing.assert_array_equal(a, b)


def test_rows_before_the_restricted_context_see_themselves_only():
    """A history row that lies before key_start attends to itself alone: its output is the single-row forward."""
    shape = synth.ModelShape(1, 32, 4, 4, 48, 40)
    w = _random_model(shape, "preverify", seed=12)
    m = orc.OracleModel(shape, w)
    rng = np.random.default_rng(4)
    rows = rng.standard_normal((3, 32))
    c = orc.Cache(m, 16)
    orc.forward(m, c, x_in=rng.standard_normal((2, 32)), want_logits=False)
    got, _ = orc.forward(m, c, x_in=rows, want_logits=False, key_start=3)     # rows at 2, 3, 4; context from 3
    single, _ = orc.forward(m, orc.Cache(m, 16), x_in=rows[:1], want_logits=False)
    np.testing.assert_allclose(got[0], single[0], atol=1e-9)
    pair, _ = orc.forward(m, orc.Cache(m, 16), x_in=rows[1:], want_logits=False)
    np.testing.assert_allclose(got[1:], pair, atol=1e-9)
