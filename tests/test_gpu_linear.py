"""Parity of the tensor-core linear layer against the fp64 reference, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import linear as ol
from paper_2504_11816_b200 import binding as B
from paper_2504_11816_b200 import workloads as W

from _harness import bits_to_dev, dev_to_bits, round_to, values

pytestmark = pytest.mark.gpu


def _case(M, N, K, dtype, seed):
    rng = np.random.default_rng(seed)
    x = W.normal_bits(rng, (M, K), dtype)
    w32 = rng.standard_normal((N, K), dtype=np.float32) / np.float32(np.sqrt(K))
    w = W._round_to_bits(w32, dtype)
    return x, w


@pytest.mark.parametrize("M,N,K,dtype", [
    (1, 128, 128, "f16"), (5, 256, 512, "f16"), (16, 128, 1024, "bf16"), (32, 512, 4096, "f16"),
    (33, 384, 2048, "bf16"), (100, 256, 1024, "f16"), (256, 256, 512, "f16"), (64, 1408, 1024, "bf16"),
    # every CTA walks more K blocks than its ring holds: wide stages (few tokens) and narrow ones (many)
    (8, 4096, 8192, "f16"), (128, 2048, 4096, "bf16"),
])
def test_linear_matches_reference(M, N, K, dtype):
    x, w = _case(M, N, K, dtype, seed=M * 7 + N)
    xd, wd = bits_to_dev(x, dtype), bits_to_dev(w, dtype)
    y32 = torch.full((M, N), float("nan"), device="cuda")
    y16 = torch.zeros((M, N), device="cuda", dtype=W.torch_dtype(dtype))
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    l = B.isv_linear_create(wd, N, K, B.ISV_F16 if dtype == "f16" else B.ISV_BF16, max(M, 16), stream.cuda_stream)
    try:
        for rep in range(2):                         # the second call meets the first one's scratch
            B.isv_linear_forward(l, xd, y16, y32, M)
            assert B.isv_linear_status(l) == 0
            ref = ol.linear(values(x, dtype), values(w, dtype))
            got = y32.cpu().numpy().astype(np.float64)
            assert np.all(np.isfinite(got))
            # fp32 accumulation of K products of magnitude ~1/sqrt(K): a few 1e-6; bound with margin
            assert np.max(np.abs(got - ref)) <= 1e-4 * max(1.0, float(np.max(np.abs(ref)))), (M, N, K, rep)
            got16 = np.asarray(values(dev_to_bits(y16), dtype).astype(np.float64) if dtype == "f16"
                               else values(dev_to_bits(y16), dtype).to(torch.float64).numpy())
            ulp = 2.0 ** -10 if dtype == "f16" else 2.0 ** -7
            assert np.max(np.abs(got16 - round_to(ref, dtype)) / np.maximum(1.0, np.abs(ref))) <= ulp
            y32.fill_(float("nan"))
    finally:
        B.isv_linear_free(l)


def test_linear_rejects_bad_shapes():
    w = torch.zeros((128, 128), device="cuda", dtype=torch.float16)
    for N, K, maxM in ((100, 128, 16), (128, 64, 16), (128, 128, 300), (0, 128, 16)):
        with pytest.raises(B.IsvError) as ei:
            B.isv_linear_create(w, N, K, B.ISV_F16, maxM, 0)
        assert ei.value.code == B.ISV_EINVAL
    l = B.isv_linear_create(w, 128, 128, B.ISV_F16, 16, 0)
    try:
        with pytest.raises(B.IsvError):
            B.isv_linear_forward(l, w, w, None, 17)
    finally:
        B.isv_linear_free(l)
