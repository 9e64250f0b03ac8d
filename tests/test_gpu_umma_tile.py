"""Self-test of the tcgen05 plumbing: one 128 x N x K bf16 tile product against a plain fp64 matrix product."""
import numpy as np
import pytest
import torch

from paper_2609_39334_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("b_mn", [0, 1])
@pytest.mark.parametrize("n,k", [(64, 64), (128, 64), (64, 128), (128, 128), (128, 256)])
def test_umma_tile_product(n, k, b_mn):
    dev = torch.device("cuda:0")
    g = torch.Generator(device="cpu").manual_seed(n * 1000 + k + b_mn)
    a = torch.randn(128, k, generator=g).to(torch.bfloat16)
    b = torch.randn((k, n) if b_mn else (n, k), generator=g).to(torch.bfloat16)
    want = a.double() @ (b.double() if b_mn else b.double().T)
    c = torch.full((128, n), float("nan"), dtype=torch.float32, device=dev)
    status = torch.full((1,), -1, dtype=torch.int32, device=dev)
    rc = B.ss_debug_umma_tile(a.to(dev), b.to(dev), c, n, k, b_mn, status)
    assert rc == B.SS_OK
    torch.cuda.synchronize()
    assert int(status.item()) == B.SS_OK
    got = c.cpu().double()
    # fp32 accumulation of exact bf16 products: error ~ k * 2^-24 * |terms|
    assert torch.isfinite(got).all()
    assert (got - want).abs().max().item() < 1e-3 * (k / 64) ** 0.5 + 1e-4


@pytest.mark.gpu
def test_bounded_wait_gives_up_and_the_kernel_ends():
    """Every role of the tensor-core kernels waits through one bounded helper; on a barrier that nothing completes it
    must return after its limit with the CTA's abort flag raised, and the context must stay usable."""
    dev = torch.device("cuda:0")
    status = torch.full((2,), -1, dtype=torch.int32, device=dev)
    assert B.ss_debug_bounded_wait(status) == B.SS_OK
    torch.cuda.synchronize()
    st = status.cpu().tolist()
    assert st[0] == B.SS_ERR_TIMEOUT
    assert 100 <= st[1] <= 4000          # ~0.2 s worth of clocks, in millions
    x = torch.arange(8, device=dev).sum().item()      # the context still works
    assert x == 28
