"""Seeded synthetic inputs for the Pacer hot path: model shapes, weights,
planted successor tables and prompts.

This module is the only thing the CPU oracle's tests and the CUDA path's tests
have in common.  It contains none of the method's arithmetic: it only turns
(seed, tensor id, element index) into numbers with integer hashing, so the same
bytes can be produced on the host or on the device, in any order and in chunks.

Every value is a pure function of its coordinates:

  weights   approximately N(0, std): the sum of eight 16-bit lanes of two
            splitmix64 hashes (an Irwin-Hall variate, exact in integers), scaled
            by ONE fp32 multiply and rounded to bf16 (round-to-nearest-even).
            All steps are exact or correctly rounded, so CPU and GPU tensors are
            bit-identical.
  succ_T    a seeded map V -> V ("planted successor"); succ_D agrees with it on
            a seeded fraction of the vocabulary and differs elsewhere.
  prompts   uniform token ids, seeded per sequence.

The synthetic pairs stand in for the pretrained model pairs and benchmark
prompts the paper measures on (Section 4.1); shapes follow Llama-style decoders.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, Optional

import torch

_MASK64 = (1 << 64) - 1


def _i64(x: int) -> int:
    """Python int -> the int64 two's-complement value with the same low 64 bits."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _i64(0x9E3779B97F4A7C15)
_M1 = _i64(0xBF58476D1CE4E5B9)
_M2 = _i64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def splitmix64(x: torch.Tensor) -> torch.Tensor:
    """The splitmix64 finaliser on an int64 tensor (wrapping arithmetic)."""
    z = x + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _splitmix64_int(x: int) -> int:
    z = (x + 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def _stream_base(seed: int, tensor_id: int) -> int:
    """A 64-bit offset that separates (seed, tensor) streams."""
    return _splitmix64_int(_splitmix64_int(seed & _MASK64) ^ ((tensor_id + 1) * 0xD1342543DE82EF95 & _MASK64))


def _lanes16_sum(h: torch.Tensor) -> torch.Tensor:
    return (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + (_lsr(h, 48) & 0xFFFF)


# std of the sum of eight independent uniform{0..65535}: sqrt(8 * (65536^2 - 1) / 12)
_IH8_STD = (8.0 * (65536.0 ** 2 - 1.0) / 12.0) ** 0.5


def normal_bf16(seed: int, tensor_id: int, shape, std: float = 0.02,
                device: str | torch.device = "cpu", chunk: int = 1 << 24) -> torch.Tensor:
    """bf16 tensor of approximately N(0, std) values, bit-identical on any device."""
    numel = 1
    for s in shape:
        numel *= int(s)
    out = torch.empty(numel, dtype=torch.bfloat16, device=device)
    base = _stream_base(seed, tensor_id)
    # (2*sum - 8*65535) is an exact integer below 2^24; one fp32 multiply follows.
    scale = torch.tensor(std / (2.0 * _IH8_STD), dtype=torch.float32).item()
    for start in range(0, numel, chunk):
        end = min(numel, start + chunk)
        idx = torch.arange(start, end, dtype=torch.int64, device=device)
        c = idx * 2 + _i64(base)
        s = _lanes16_sum(splitmix64(c)) + _lanes16_sum(splitmix64(c + 1))
        v = (2 * s - 8 * 65535).to(torch.float32) * scale
        out[start:end] = v.to(torch.bfloat16)
    return out.view(*shape)


def hashed_ints(seed: int, tensor_id: int, n: int, modulo: int, device="cpu") -> torch.Tensor:
    """int64 tensor of n seeded values in [0, modulo)."""
    base = _stream_base(seed, tensor_id)
    idx = torch.arange(n, dtype=torch.int64, device=device)
    h = splitmix64(idx + _i64(base))
    return _lsr(h, 1) % modulo


# --------------------------------------------------------------------------------------
# shapes
# --------------------------------------------------------------------------------------

@dataclasses.dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    d_ffn: int
    vocab: int
    rope_theta: float = 10000.0
    rms_eps: float = 1e-5

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_heads

    @property
    def qkv_rows(self) -> int:
        return (self.n_heads + 2 * self.n_kv_heads) * self.head_dim

    def n_params(self) -> int:
        per_layer = (self.qkv_rows * self.d_model + self.d_model * self.n_heads * self.head_dim
                     + 3 * self.d_model * self.d_ffn)
        return self.n_layers * per_layer + 2 * self.vocab * self.d_model

    def streamed_weight_bytes(self) -> int:
        """bf16 bytes one forward must read: all layer matrices and the LM head
        (the embedding table is gathered, not streamed)."""
        per_layer = (self.qkv_rows * self.d_model + self.d_model * self.n_heads * self.head_dim
                     + 3 * self.d_model * self.d_ffn)
        return 2 * (self.n_layers * per_layer + self.vocab * self.d_model)

    def kv_bytes_per_token(self) -> int:
        return 2 * self.n_layers * self.n_kv_heads * self.head_dim * 2


@dataclasses.dataclass(frozen=True)
class PairConfig:
    name: str
    target: ModelShape
    draft: ModelShape
    agree: float            # fraction of the vocabulary on which succ_D == succ_T
    n_prompt: int
    max_new: int
    gamma_max: int
    batch: int = 1
    block_b: int = 4
    rho: float = 1.05
    succ_bias: float = 8.0

    @property
    def gamma_cap(self) -> int:
        return (self.gamma_max // self.block_b) * self.block_b


_D68M = ModelShape(2, 768, 12, 12, 3072, 32000)

CONFIGS: Dict[str, PairConfig] = {
    "tiny": PairConfig("tiny", ModelShape(4, 256, 4, 4, 1024, 4096), ModelShape(1, 128, 2, 2, 512, 4096),
                       agree=0.80, n_prompt=64, max_new=64, gamma_max=8),
    "7b_68m": PairConfig("7b_68m", ModelShape(32, 4096, 32, 32, 11008, 32000), _D68M,
                         agree=0.80, n_prompt=512, max_new=256, gamma_max=16),
    "13b_68m": PairConfig("13b_68m", ModelShape(40, 5120, 40, 40, 13824, 32000), _D68M,
                          agree=0.65, n_prompt=1024, max_new=512, gamma_max=16),
    "33b_1b3": PairConfig("33b_1b3", ModelShape(62, 7168, 56, 8, 19200, 32256),
                          ModelShape(24, 2048, 16, 16, 5504, 32256),
                          agree=0.85, n_prompt=2048, max_new=512, gamma_max=24),
    # a second workload: grouped-query models with a large vocabulary (the shapes of a 1.5B / 32B pair of the
    # Qwen2.5 family, the other family the paper measures): the draft's LM head is a fifth of its weights
    "qwen_32b_1b5": PairConfig("qwen_32b_1b5", ModelShape(64, 5120, 40, 8, 27648, 151936),
                               ModelShape(28, 1536, 12, 2, 8960, 151936),
                               agree=0.80, n_prompt=1024, max_new=256, gamma_max=16),
    "7b_68m_long_b8": PairConfig("7b_68m_long_b8", ModelShape(32, 4096, 32, 32, 11008, 32000), _D68M,
                                 agree=0.80, n_prompt=8192, max_new=256, gamma_max=16, batch=8),
}

# tensor kinds; the index is part of the hash stream id
_KINDS = ("embed", "wqkv", "wo", "wgate", "wup", "wdown", "norm1", "norm2", "normf", "head",
          "head_b", "posemb")
_WHICH = {"target": 0, "draft": 1, "preverify": 2}
_ID_SUCC_T, _ID_SUCC_D_PICK, _ID_SUCC_D_ALT, _ID_PROMPT = 900, 901, 902, 1000


def model_tensor_shapes(shape: ModelShape, which: str, gamma_cap: int = 0) -> Dict[str, tuple]:
    """Name -> shape of every tensor of one model.  Matrices are [out][in]
    row-major, stacked over layers; q, k, v rows are stacked in that order."""
    L, d, F, V = shape.n_layers, shape.d_model, shape.d_ffn, shape.vocab
    t = {
        "wqkv": (L, shape.qkv_rows, d),
        "wo": (L, d, shape.n_heads * shape.head_dim),
        "wgate": (L, F, d),
        "wup": (L, F, d),
        "wdown": (L, d, F),
        "norm1": (L, d),
        "norm2": (L, d),
        "normf": (d,),
    }
    if which == "preverify":
        t["head_b"] = (2, d)
        t["posemb"] = (gamma_cap, d)
    else:
        t["embed"] = (V, d)
        t["head"] = (V, d)
    return t


def make_model(shape: ModelShape, which: str, seed: int = 0, device="cpu", gamma_cap: int = 0,
               std: float = 0.02) -> Dict[str, torch.Tensor]:
    """All tensors of one model as bf16: matrices ~ N(0, std), norm gains 1."""
    out = {}
    for name, shp in model_tensor_shapes(shape, which, gamma_cap).items():
        if name.startswith("norm"):
            out[name] = torch.ones(shp, dtype=torch.bfloat16, device=device)
        else:
            tid = _WHICH[which] * 32 + _KINDS.index(name)
            out[name] = normal_bf16(seed, tid, shp, std=std, device=device)
    return out


def preverify_shape(draft: ModelShape) -> ModelShape:
    """The pre-verification layer: ONE decoder layer with the draft's widths."""
    return dataclasses.replace(draft, n_layers=1)


def make_succ_tables(vocab: int, agree: float, seed: int = 0, device="cpu"):
    """(succ_T, succ_D) int32[V].  succ_D[v] == succ_T[v] on a seeded fraction
    `agree` of v and is a different token elsewhere."""
    succ_t = hashed_ints(seed, _ID_SUCC_T, vocab, vocab, device)
    pick = hashed_ints(seed, _ID_SUCC_D_PICK, vocab, 1 << 20, device)
    alt = hashed_ints(seed, _ID_SUCC_D_ALT, vocab, max(vocab - 1, 1), device)
    other = (succ_t + 1 + alt) % vocab
    succ_d = torch.where(pick < int(agree * (1 << 20)), succ_t, other)
    return succ_t.to(torch.int32), succ_d.to(torch.int32)


def make_prompts(vocab: int, batch: int, n_prompt: int, seed: int = 0) -> torch.Tensor:
    """int32 [batch][n_prompt] uniform token ids on the host, seeded per sequence."""
    rows = [hashed_ints(seed, _ID_PROMPT + s, n_prompt, vocab) for s in range(batch)]
    return torch.stack(rows).to(torch.int32)


def make_pair(cfg: PairConfig, seed: int = 0, device="cpu",
              which=("target", "draft", "preverify"), std: float = 0.02) -> Dict[str, Optional[dict]]:
    """Weights of the requested models of a pair plus the successor tables."""
    out: Dict[str, Optional[dict]] = {}
    if "target" in which:
        out["target"] = make_model(cfg.target, "target", seed, device, std=std)
    if "draft" in which:
        out["draft"] = make_model(cfg.draft, "draft", seed, device, std=std)
    if "preverify" in which:
        out["preverify"] = make_model(preverify_shape(cfg.draft), "preverify", seed, device,
                                      gamma_cap=cfg.gamma_cap, std=std)
    st, sd = make_succ_tables(cfg.target.vocab, cfg.agree, seed, device)
    out["succ_T"], out["succ_D"] = st, sd
    return out
