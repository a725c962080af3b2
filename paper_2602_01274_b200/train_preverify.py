"""Trains the pre-verification layer M_B for a synthetic pair with the paper's recipe.

Section 3.3 and the appendix on training details: the target model generates a
response to every prompt; from every prefix of that response the draft model
drafts gamma tokens; draft token i is labelled 1 while it and all drafts before
it equal the target's tokens at their positions, 0 from the first mismatch on;
M_B sees the draft's hidden states ([h_i + e_i] for the drafts, the plain hidden
states of the prefix as history) and is trained with cross-entropy on the
labels, AdamW (0.9, 0.999).  All draft steps of one prompt share the prefix rows
(the packed attention mask of the appendix): a draft row attends to the prefix
rows before its own start and to the drafts of its own step.

This is a small PyTorch job OUTSIDE the decoding path: it produces the bf16
tensors `pacer_load_weights(PACER_PREVERIFY, ...)` takes (and the CPU oracle
reads), nothing more.  It needs no dataset: prompts are seeded random tokens and
the responses come from the synthetic target.  The window used for the labels is
gamma_cap (the position-embedding table has that many rows), not the paper's 50.

    python -m paper_2602_01274_b200.train_preverify --config 7b_68m --out mb_7b.pt
"""
from __future__ import annotations

import argparse
import math
import time
from typing import Dict

import torch
import torch.nn.functional as F

from . import synth


# ----------------------------------------------------------------------------- plain torch decoder (data generation)

def _rope_tables(shape, n_pos, device):
    hd = shape.head_dim
    inv = shape.rope_theta ** (-torch.arange(0, hd // 2, dtype=torch.float64, device=device) * 2.0 / hd)
    ang = torch.arange(n_pos, dtype=torch.float64, device=device)[:, None] * inv[None, :]
    return ang.cos().float(), ang.sin().float()


def _rope(t, cos, sin, pos):
    """t [..., n, heads, hd]; pos [..., n] absolute positions (long)."""
    half = t.shape[-1] // 2
    c, s = cos[pos][..., None, :], sin[pos][..., None, :]
    a, b = t[..., :half], t[..., half:]
    return torch.cat([a * c - b * s, b * c + a * s], dim=-1)


def _rms(x, g, eps):
    return x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + eps) * g


class Decoder:
    """Llama-style decoder in plain torch with a KV cache, batch-first, for generating training data."""

    def __init__(self, shape, w: Dict[str, torch.Tensor], succ, succ_bias, max_pos, dtype=torch.float32):
        self.s, self.succ, self.bias, self.dt = shape, succ.long() if succ is not None else None, succ_bias, dtype
        self.w = {k: v.to(dtype) for k, v in w.items()}
        self.cos, self.sin = _rope_tables(shape, max_pos, next(iter(w.values())).device)
        self.k = self.v = None

    def reset(self, batch, max_len):
        s = self.s
        dev = self.w["wqkv"].device
        self.k = torch.zeros(s.n_layers, batch, max_len, s.n_kv_heads, s.head_dim, dtype=self.dt, device=dev)
        self.v = torch.zeros_like(self.k)
        self.len = 0

    @torch.no_grad()
    def forward(self, tokens):
        """tokens [B][n] appended at positions len..len+n-1; returns (hidden [B][n][d] fp32, logits [B][n][V] fp32)."""
        s, w = self.s, self.w
        B, n = tokens.shape
        H, Hkv, hd = s.n_heads, s.n_kv_heads, s.head_dim
        pos = torch.arange(self.len, self.len + n, device=tokens.device)
        x = w["embed"][tokens].float()
        for l in range(s.n_layers):
            a = _rms(x, w["norm1"][l].float(), s.rms_eps).to(self.dt)
            qkv = (a @ w["wqkv"][l].T).float()
            q = _rope(qkv[..., : H * hd].view(B, n, H, hd), self.cos, self.sin, pos)
            k = _rope(qkv[..., H * hd: (H + Hkv) * hd].view(B, n, Hkv, hd), self.cos, self.sin, pos)
            v = qkv[..., (H + Hkv) * hd:].view(B, n, Hkv, hd)
            self.k[l, :, self.len: self.len + n] = k.to(self.dt)
            self.v[l, :, self.len: self.len + n] = v.to(self.dt)
            T = self.len + n
            kk = self.k[l, :, :T].float().repeat_interleave(H // Hkv, dim=2)
            vv = self.v[l, :, :T].float().repeat_interleave(H // Hkv, dim=2)
            mask = (torch.arange(T, device=x.device)[None, :] <= pos[:, None])          # [n][T]
            att = F.scaled_dot_product_attention(q.transpose(1, 2), kk.transpose(1, 2), vv.transpose(1, 2), attn_mask=mask)
            x = x + (att.transpose(1, 2).reshape(B, n, H * hd).to(self.dt) @ w["wo"][l].T).float()
            m = _rms(x, w["norm2"][l].float(), s.rms_eps).to(self.dt)
            x = x + ((F.silu((m @ w["wgate"][l].T).float()) * (m @ w["wup"][l].T).float()).to(self.dt) @ w["wdown"][l].T).float()
        self.len += n
        hid = _rms(x, w["normf"].float(), s.rms_eps)
        logits = (hid.to(self.dt) @ w["head"].T).float()
        if self.succ is not None:
            logits.scatter_add_(2, self.succ[tokens][..., None], torch.full((B, n, 1), float(self.bias), device=x.device))
        return hid, logits


# ----------------------------------------------------------------------------- data: drafts from every prefix

@torch.no_grad()
def make_examples(cfg: synth.PairConfig, pair, prompts, n_resp, gamma, dtype, prefix_stride=1):
    """For a batch of prompts [B][n_p]: the target's greedy response (n_resp tokens), then from every prefix end
    p = n_p-1, n_p-1+stride, ... gamma greedy drafts.  Returns a dict of tensors:
      hist   [B][T][d]      draft hidden state of every sequence position (the history rows of M_B), T = n_p + n_resp
      h      [B][R][g][d]   hidden state of the forward that emitted draft m of prefix r
      label  [B][R][g]      1 while the drafts match the target's tokens, 0 from the first mismatch on
      valid  [B][R][g]      0 where the target's token at that position is unknown (past the response)
      p      [R]            prefix end positions"""
    dev = prompts.device
    B, n_p = prompts.shape
    T = n_p + n_resp
    tgt = Decoder(cfg.target, pair["target"], pair["succ_T"], cfg.succ_bias, T + 1, dtype)
    tgt.reset(B, T)
    _, lg = tgt.forward(prompts)
    seq = [prompts]
    nxt = lg[:, -1].argmax(-1, keepdim=True)
    for _ in range(n_resp):
        seq.append(nxt)
        if len(seq) - 1 == n_resp:
            break
        _, lg = tgt.forward(nxt)
        nxt = lg[:, -1].argmax(-1, keepdim=True)
    full = torch.cat(seq, dim=1)                                    # [B][T]
    del tgt

    ds, dw = cfg.draft, {k: v.to(dtype) for k, v in pair["draft"].items()}
    drf = Decoder(ds, pair["draft"], pair["succ_D"], cfg.succ_bias, T + gamma + 1, dtype)
    drf.reset(B, T)
    hist, dlg = drf.forward(full)                                   # teacher-forced pass: history rows and first drafts
    P = torch.arange(n_p - 1, T - 1, prefix_stride, device=dev)     # prefix end positions (the last accepted token)
    R = P.numel()
    H, Hkv, hd, L = ds.n_heads, ds.n_kv_heads, ds.head_dim, ds.n_layers
    h = torch.zeros(B, R, gamma, ds.d_model, device=dev)
    d_tok = torch.zeros(B, R, gamma, dtype=torch.long, device=dev)
    h[:, :, 0] = hist[:, P]
    d_tok[:, :, 0] = dlg[:, P].argmax(-1)
    ok = torch.ones(B, R, gamma, dtype=torch.bool, device=dev)
    own_k = torch.zeros(L, B, R, gamma, Hkv, hd, device=dev, dtype=dtype)
    own_v = torch.zeros_like(own_k)
    cos, sin = drf.cos, drf.sin
    t_idx = torch.arange(T, device=dev)
    pre_mask = (t_idx[None, :] <= P[:, None])                       # [R][T]: prefix keys a step may see
    succ = pair["succ_D"].long()
    for m in range(1, gamma):                                       # draft m+1 from input d_m at position p + m
        tok_in = d_tok[:, :, m - 1]                                 # [B][R]
        pos = (P + m)[None, :].expand(B, R)
        x = dw["embed"][tok_in].float()
        for l in range(L):
            a = _rms(x, dw["norm1"][l].float(), ds.rms_eps).to(dtype)
            qkv = (a @ dw["wqkv"][l].T).float()
            q = _rope(qkv[..., : H * hd].view(B, R, 1, H, hd), cos, sin, pos[..., None])[:, :, 0]          # [B][R][H][hd]
            k = _rope(qkv[..., H * hd: (H + Hkv) * hd].view(B, R, 1, Hkv, hd), cos, sin, pos[..., None])[:, :, 0]
            v = qkv[..., (H + Hkv) * hd:].view(B, R, Hkv, hd)
            own_k[l, :, :, m - 1] = k.to(dtype)
            own_v[l, :, :, m - 1] = v.to(dtype)
            g = H // Hkv
            qg = q.view(B, R, Hkv, g, hd)
            s_pre = torch.einsum("brkgd,btkd->brkgt", qg, drf.k[l].float()) / math.sqrt(hd)
            s_pre = s_pre.masked_fill(~pre_mask[None, :, None, None, :], float("-inf"))
            s_own = torch.einsum("brkgd,brmkd->brkgm", qg, own_k[l, :, :, :m].float()) / math.sqrt(hd)
            pr = torch.softmax(torch.cat([s_pre, s_own], dim=-1), dim=-1)
            att = torch.einsum("brkgt,btkd->brkgd", pr[..., :T], drf.v[l].float()) + \
                torch.einsum("brkgm,brmkd->brkgd", pr[..., T:], own_v[l, :, :, :m].float())
            x = x + (att.reshape(B, R, H * hd).to(dtype) @ dw["wo"][l].T).float()
            mm = _rms(x, dw["norm2"][l].float(), ds.rms_eps).to(dtype)
            x = x + ((F.silu((mm @ dw["wgate"][l].T).float()) * (mm @ dw["wup"][l].T).float()).to(dtype) @ dw["wdown"][l].T).float()
        hid = _rms(x, dw["normf"].float(), ds.rms_eps)
        lgt = (hid.to(dtype) @ dw["head"].T).float()
        lgt.scatter_add_(2, succ[tok_in][..., None], torch.full((B, R, 1), float(cfg.succ_bias), device=dev))
        h[:, :, m] = hid
        d_tok[:, :, m] = lgt.argmax(-1)
    # labels: draft m (0-based) of prefix p is the candidate for position p + 1 + m
    tpos = P[:, None] + 1 + torch.arange(gamma, device=dev)[None, :]                                      # [R][g]
    valid = (tpos < T)[None].expand(B, R, gamma)
    want = full[:, tpos.clamp(max=T - 1)]                                                                  # [B][R][g]
    match = (d_tok == want) & valid
    label = torch.cumprod(match.long(), dim=-1)
    return dict(hist=hist, h=h, label=label, valid=valid & ok, p=P, tokens=full, drafts=d_tok)


# ----------------------------------------------------------------------------- M_B in torch (training forward)

class PreVerify(torch.nn.Module):
    """One decoder layer at draft width + RMSNorm + Linear(d -> 2), with the draft position embedding table
    (Eq. 7; the same tensors and layout pacer_load_weights takes for the pre-verification model)."""

    def __init__(self, shape, gamma_cap, seed=0):
        super().__init__()
        self.s = synth.preverify_shape(shape)
        d, F_, s = shape.d_model, shape.d_ffn, self.s
        g = torch.Generator().manual_seed(seed)
        rnd = lambda *sz: torch.nn.Parameter(torch.randn(*sz, generator=g) * 0.02)
        self.wqkv, self.wo = rnd(1, s.qkv_rows, d), rnd(1, d, s.n_heads * s.head_dim)
        self.wgate, self.wup, self.wdown = rnd(1, F_, d), rnd(1, F_, d), rnd(1, d, F_)
        self.norm1, self.norm2 = torch.nn.Parameter(torch.ones(1, d)), torch.nn.Parameter(torch.ones(1, d))
        self.normf = torch.nn.Parameter(torch.ones(d))
        self.head_b, self.posemb = rnd(2, d), rnd(gamma_cap, d)

    def forward(self, hist, h, P, use_posemb=True):
        """hist [B][T][d], h [B][R][g][d], P [R] -> logits [B][R][g][2].  Draft row m of prefix r sits at position
        P[r] + m and attends to the history rows 0..P[r]-1 and to the drafts 0..m of its own step."""
        s = self.s
        B, R, g, d = h.shape
        T = hist.shape[1]
        H, Hkv, hd = s.n_heads, s.n_kv_heads, s.head_dim
        dev = h.device
        cos, sin = _rope_tables(s, T + g + 1, dev)
        x = h + (self.posemb[None, None, :g] if use_posemb else 0.0)
        # history rows: only their keys and values matter (one layer)
        ah = _rms(hist, self.norm1[0], s.rms_eps)
        qkv_h = ah @ self.wqkv[0].T
        pos_h = torch.arange(T, device=dev)[None].expand(B, T)
        k_h = _rope(qkv_h[..., H * hd: (H + Hkv) * hd].view(B, T, Hkv, hd), cos, sin, pos_h)
        v_h = qkv_h[..., (H + Hkv) * hd:].view(B, T, Hkv, hd)
        a = _rms(x, self.norm1[0], s.rms_eps)
        qkv = a @ self.wqkv[0].T
        pos = (P[:, None] + torch.arange(g, device=dev)[None, :])[None].expand(B, R, g)
        q = _rope(qkv[..., : H * hd].view(B, R, g, H, hd), cos, sin, pos)
        k = _rope(qkv[..., H * hd: (H + Hkv) * hd].view(B, R, g, Hkv, hd), cos, sin, pos)
        v = qkv[..., (H + Hkv) * hd:].view(B, R, g, Hkv, hd)
        grp = H // Hkv
        qg = q.view(B, R, g, Hkv, grp, hd)
        s_h = torch.einsum("brmkgd,btkd->brmkgt", qg, k_h) / math.sqrt(hd)
        hmask = torch.arange(T, device=dev)[None, :] < P[:, None]                         # [R][T]
        s_h = s_h.masked_fill(~hmask[None, :, None, None, None, :], float("-inf"))
        s_o = torch.einsum("brmkgd,brnkd->brmkgn", qg, k) / math.sqrt(hd)
        cmask = torch.tril(torch.ones(g, g, dtype=torch.bool, device=dev))                # [m][n]: n <= m
        s_o = s_o.masked_fill(~cmask[None, None, :, None, None, :], float("-inf"))
        pr = torch.softmax(torch.cat([s_h, s_o], dim=-1), dim=-1)
        att = torch.einsum("brmkgt,btkd->brmkgd", pr[..., :T], v_h) + torch.einsum("brmkgn,brnkd->brmkgd", pr[..., T:], v)
        x = x + att.reshape(B, R, g, H * hd) @ self.wo[0].T
        mm = _rms(x, self.norm2[0], s.rms_eps)
        x = x + (F.silu(mm @ self.wgate[0].T) * (mm @ self.wup[0].T)) @ self.wdown[0].T
        return _rms(x, self.normf, s.rms_eps) @ self.head_b.T

    def export(self) -> Dict[str, torch.Tensor]:
        """bf16 tensors under the names pacer_load_weights expects."""
        return {k: getattr(self, k).detach().to(torch.bfloat16).contiguous()
                for k in ("wqkv", "wo", "wgate", "wup", "wdown", "norm1", "norm2", "normf", "head_b", "posemb")}


def auc(score, label):
    """Area under the ROC curve (probability that a positive outranks a negative)."""
    score, label = score.flatten().double(), label.flatten().bool()
    n1, n0 = int(label.sum()), int((~label).sum())
    if n1 == 0 or n0 == 0:
        return float("nan")
    order = score.argsort()
    ranks = torch.empty_like(score)
    ranks[order] = torch.arange(1, score.numel() + 1, dtype=torch.float64, device=score.device)
    return float((ranks[label].sum() - n1 * (n1 + 1) / 2) / (n1 * n0))


def train(cfg: synth.PairConfig, pair, device="cpu", n_prompts=64, n_prompt_tokens=32, n_resp=96, epochs=5, lr=5e-4,
          batch_prompts=8, prefix_stride=1, seed=0, dtype=None, log=print, prompt_seed=1000):
    """Returns (bf16 tensors of the trained M_B, report dict).  `pair` holds the target and draft tensors on `device`."""
    dtype = dtype or (torch.bfloat16 if str(device).startswith("cuda") else torch.float32)
    gamma = cfg.gamma_cap
    t0 = time.time()
    data = []
    for i in range(0, n_prompts + batch_prompts, batch_prompts):      # the last batch is held out
        prompts = synth.make_prompts(cfg.target.vocab, batch_prompts, n_prompt_tokens, seed=prompt_seed + i).to(device).long()
        data.append(make_examples(cfg, pair, prompts, n_resp, gamma, dtype, prefix_stride))
    held = data.pop()
    base = float(torch.cat([d["label"][d["valid"]].float() for d in data]).mean())
    log(f"[train_preverify] {len(data)} batches of {batch_prompts} prompts in {time.time() - t0:.1f} s; "
        f"share of accepted labels {base:.3f}")
    torch.manual_seed(seed)
    mb = PreVerify(cfg.draft, gamma, seed).to(device)
    opt = torch.optim.AdamW(mb.parameters(), lr=lr, betas=(0.9, 0.999))
    steps = epochs * len(data)
    sched = torch.optim.lr_scheduler.OneCycleLR(opt, max_lr=lr, total_steps=max(steps, 2), pct_start=0.1)
    for ep in range(epochs):
        tot = n = 0.0
        for di in torch.randperm(len(data), generator=torch.Generator().manual_seed(seed + ep)).tolist():
            d = data[di]
            lg = mb(d["hist"], d["h"], d["p"])
            loss = F.cross_entropy(lg[d["valid"]], d["label"][d["valid"]])
            opt.zero_grad(set_to_none=True)
            loss.backward()
            opt.step(); sched.step()
            tot += float(loss.detach()); n += 1
        log(f"[train_preverify] epoch {ep + 1}/{epochs}: loss {tot / n:.4f}")
    with torch.no_grad():
        lg = mb(held["hist"], held["h"], held["p"])
        sc = torch.softmax(lg, -1)[..., 1][held["valid"]]
        lb = held["label"][held["valid"]]
        rep = {"held_out_auc": auc(sc, lb), "held_out_loss": float(F.cross_entropy(lg[held["valid"]], lb)),
               "held_out_accept_share": float(lb.float().mean()), "train_accept_share": base,
               "mean_alpha_accepted": float(sc[lb == 1].mean()) if (lb == 1).any() else float("nan"),
               "mean_alpha_rejected": float(sc[lb == 0].mean()) if (lb == 0).any() else float("nan"),
               "prompts": n_prompts, "response_tokens": n_resp, "epochs": epochs, "lr": lr, "window": gamma,
               "seconds": time.time() - t0}
    log(f"[train_preverify] held-out AUC {rep['held_out_auc']:.3f}, alpha_hat accepted {rep['mean_alpha_accepted']:.3f} / "
        f"rejected {rep['mean_alpha_rejected']:.3f}")
    return mb.export(), rep


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="tiny")
    ap.add_argument("--out", required=True)
    ap.add_argument("--device", default="cuda:0" if torch.cuda.is_available() else "cpu")
    ap.add_argument("--prompts", type=int, default=64)
    ap.add_argument("--prompt-tokens", type=int, default=32)
    ap.add_argument("--response-tokens", type=int, default=96)
    ap.add_argument("--epochs", type=int, default=5)
    ap.add_argument("--lr", type=float, default=5e-4)
    ap.add_argument("--batch-prompts", type=int, default=8)
    args = ap.parse_args()
    cfg = synth.CONFIGS[args.config]
    pair = synth.make_pair(cfg, seed=0, device=args.device, which=("target", "draft"))
    w, rep = train(cfg, pair, args.device, args.prompts, args.prompt_tokens, args.response_tokens, args.epochs, args.lr,
                   batch_prompts=args.batch_prompts)
    torch.save({"tensors": {k: v.cpu() for k, v in w.items()}, "report": rep, "config": args.config}, args.out)
    print(rep)


if __name__ == "__main__":
    main()
