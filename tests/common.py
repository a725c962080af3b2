"""Helpers shared by the tests: build oracle models from the seeded inputs."""
import dataclasses

import torch

from oracle import pacer_oracle as orc
from paper_2602_01274_b200 import synth


def oracle_models(cfg: synth.PairConfig, pair: dict, fp32: bool = False):
    """(T, D, B) OracleModel objects reading the given pair's tensors (moved to the host)."""
    def conv(d):
        out = {k: v.detach().cpu() for k, v in d.items()}
        if fp32:
            out = {k: v.float() for k, v in out.items()}
        return out
    T = orc.OracleModel(cfg.target, conv(pair["target"]), pair["succ_T"], cfg.succ_bias)
    D = orc.OracleModel(cfg.draft, conv(pair["draft"]), pair["succ_D"], cfg.succ_bias)
    B = None
    if pair.get("preverify") is not None:
        B = orc.OracleModel(synth.preverify_shape(cfg.draft), conv(pair["preverify"]))
    return T, D, B


def small_pair_config(vocab=64, d_t=32, d_d=16, layers_t=2, agree=0.7, gamma_max=8, b=4, kv_t=None):
    """A pair far smaller than the tiny config, for loops that run thousands of times."""
    t = synth.ModelShape(layers_t, d_t, 4, kv_t or 4, 2 * d_t, vocab)
    d = synth.ModelShape(1, d_d, 2, 2, 2 * d_d, vocab)
    return synth.PairConfig("small", t, d, agree=agree, n_prompt=8, max_new=24, gamma_max=gamma_max, block_b=b)
