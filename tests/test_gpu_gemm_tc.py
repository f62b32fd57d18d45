"""The tensor-core projection for many shared-weight rows (tcgen05.mma, accumulator in tensor memory)
against a float64 matrix product of the same bf16-rounded operands.

fp32 accumulation of K <= 3072 products of magnitude ~|w||a| differs from the float64 sum by at most
~K * 2^-24 relative to sum |w a|; the bound used below is 2e-6 * sum_k |w a| + 1e-6, checked element-wise."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(rows, K, n, seed):
    g = torch.Generator().manual_seed(seed)
    w = (torch.randn((rows, K), generator=g) * 0.05).to(torch.bfloat16)
    a = torch.randn((n, K), generator=g)
    return w, a


@pytest.mark.parametrize("rows,K,n,ks", [(128, 128, 16, 1), (256, 256, 96, 1), (768, 768, 96, 3), (2304, 768, 96, 6),
                                         (384, 200, 5, 1), (768, 3072, 128, 24), (1000, 768, 33, 2), (768, 768, 192, 6), (256, 384, 256, 1)])
def test_gemm_tc_matches_float64_product(rows, K, n, ks):
    from paper_2601_20357_b200 import binding as TB
    dev = torch.device("cuda", 0)
    w, a = _case(rows, K, n, 1000 + rows + K + n)
    out = TB.debug_gemm_tc(w.to(dev), a.to(dev).contiguous(), ks)
    torch.cuda.synchronize()
    a16 = a.to(torch.bfloat16).double()
    ref = a16 @ w.double().T
    bound = 2e-6 * (a16.abs() @ w.double().abs().T) + 1e-6
    err = (out.cpu().double() - ref).abs()
    assert bool((err <= bound).all()), f"max err {err.max().item()} (bound {bound.max().item()})"


def test_gemm_tc_rejects_bad_sizes():
    from paper_2601_20357_b200 import binding as TB
    dev = torch.device("cuda", 0)
    w, a = _case(128, 132, 4, 7)
    with pytest.raises(TB.TabedError):
        TB.debug_gemm_tc(w.to(dev), a.to(dev), 1)          # K not a multiple of 8
    w, a = _case(128, 128, 300, 7)
    with pytest.raises(TB.TabedError):
        TB.debug_gemm_tc(w.to(dev), a.to(dev), 1)          # more than 256 slots per launch
