"""The allocation-free product entry point against the ordinary one.

pacer_linear_static serves callers that cannot hand the library any scratch memory (a server whose arena owns
the whole device, a host without an allocator): its scratch is a fixed array inside the library.  The check:
through the C ABI, twice in a row on different inputs and shapes (the array keeps the first call's contents),
its output must equal pacer_linear's, which gets fresh caller scratch.  Both run the same kernels in the same
order, so the comparison is exact; the tolerance of the other product tests is kept as the stated bound.  The
same output is also compared with the CPU oracle's product on sampled columns."""
import numpy as np
import pytest
import torch

from oracle import pacer_oracle as orc
from paper_2602_01274_b200 import synth

pytestmark = pytest.mark.gpu


def test_static_scratch_product_equals_the_ordinary_one_twice_in_a_row():
    from paper_2602_01274_b200 import binding as b
    dev = "cuda:0"
    for i, (rows, N, K) in enumerate([(17, 4096, 4096), (5, 2304, 768)]):
        w = synth.normal_bf16(7 + i, 21, (N, K), std=0.02, device=dev)
        x = synth.normal_bf16(8 + i, 22, (rows, K), std=1.0, device=dev)
        ref = b.pacer_linear(x, w)
        out = torch.full((rows, N), float("nan"), dtype=torch.float32, device=dev)   # allocated by the caller
        b.pacer_linear_static(x, w, out)
        torch.cuda.synchronize()
        err = (out - ref).abs().max().item()
        assert err <= 2e-4 * max(1.0, ref.abs().max().item()), (i, err)
        # and against the CPU oracle's product on sampled output columns, like the ordinary entry point's own test
        cols = np.unique(np.concatenate([np.arange(24), np.arange(N - 24, N), np.random.default_rng(N + K).integers(0, N, 200)]))
        want = orc.linear(w[torch.as_tensor(cols, device=dev)].cpu(), x.float().cpu().double().numpy())
        err_o = np.abs(out[:, torch.as_tensor(cols, device=dev)].cpu().double().numpy() - want).max()
        assert err_o <= 2e-4 * max(1.0, np.abs(want).max()), (i, err_o)


def test_static_scratch_product_refuses_shapes_beyond_its_array():
    from paper_2602_01274_b200 import binding as b
    dev = "cuda:0"
    rows, N, K = 32, 32000, 4096          # needs about 8 MB of partial sums
    assert b._lib.pacer_linear_scratch_bytes(rows, N, K) > b.PACER_LINEAR_STATIC_BYTES
    x = torch.zeros(rows, K, dtype=torch.bfloat16, device=dev)
    w = torch.zeros(N, K, dtype=torch.bfloat16, device=dev)
    out = torch.zeros(rows, N, dtype=torch.float32, device=dev)
    with pytest.raises(b.PacerError):
        b.pacer_linear_static(x, w, out)
