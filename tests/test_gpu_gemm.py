"""GPU check of the tensor-core batched bf16 product (lsgd_bgemm_bf16) against a library matmul:
exact equality on small-integer operands (every partial sum is exactly representable in fp32), a
tolerance on normal operands, every operand-major combination, ragged tiles, batching, epilogues."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _run(api, torch, A, B, M, N, K, batch, a_mn, b_mn, epilogue=0, bias=None, mask=None, share_a=False):
    out_dtype = torch.float32 if epilogue == 0 else torch.bfloat16
    Cmat = torch.full((batch, M, N), float("nan"), device="cuda", dtype=out_dtype)
    d = api.BgemmDesc()
    d.a, d.b, d.c = A.data_ptr(), B.data_ptr(), Cmat.data_ptr()
    d.M, d.N, d.K, d.batch = M, N, K, batch
    d.a_mn_major, d.b_mn_major = int(a_mn), int(b_mn)
    d.lda = A.shape[-1]
    d.ldb = B.shape[-1]
    d.ldc = N
    d.stride_a = 0 if share_a else A.shape[-2] * A.shape[-1]
    d.stride_b = B.shape[-2] * B.shape[-1]
    d.stride_c = M * N
    d.epilogue = epilogue
    if bias is not None:
        d.bias, d.stride_bias = bias.data_ptr(), N
    if mask is not None:
        d.mask, d.ld_mask, d.stride_mask = mask.data_ptr(), N, M * N
    api.lsgd_bgemm_bf16(d, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return Cmat


def _operands(torch, gen, M, N, K, batch, a_mn, b_mn, integer, share_a=False):
    def draw(*shape):
        if integer:
            return torch.randint(-2, 3, shape, generator=gen, device="cuda").to(torch.bfloat16)
        return torch.randn(shape, generator=gen, device="cuda").to(torch.bfloat16)
    ba = 1 if share_a else batch
    A = draw(ba, K, M) if a_mn else draw(ba, M, K)
    B = draw(batch, K, N) if b_mn else draw(batch, N, K)
    Am = (A.transpose(1, 2) if a_mn else A).double()          # [b, M, K]
    Bm = (B.transpose(1, 2) if b_mn else B).double()          # [b, N, K]
    ref = Am @ Bm.transpose(1, 2)
    return A, B, ref


SHAPES = [(128, 128, 64, 1), (128, 256, 192, 2), (200, 136, 72, 3), (256, 784, 128, 2), (128, 1024, 784, 2),
          (1024, 1024, 128, 1), (8, 8, 8, 1)]


@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_bgemm_exact_on_integer_operands(a_mn, b_mn):
    import torch
    from paper_1905_10395_b200 import api
    gen = torch.Generator(device="cuda").manual_seed(1234 + 2 * a_mn + b_mn)
    for (M, N, K, batch) in SHAPES:
        A, B, ref = _operands(torch, gen, M, N, K, batch, a_mn, b_mn, integer=True)
        got = _run(api, torch, A, B, M, N, K, batch, a_mn, b_mn)
        assert torch.equal(got.double(), ref), (M, N, K, batch, a_mn, b_mn, (got.double() - ref).abs().max().item())


@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_bgemm_normal_operands_within_fp32_accumulation_error(a_mn, b_mn):
    import torch
    from paper_1905_10395_b200 import api
    gen = torch.Generator(device="cuda").manual_seed(99 + 2 * a_mn + b_mn)
    for (M, N, K, batch) in SHAPES:
        A, B, ref = _operands(torch, gen, M, N, K, batch, a_mn, b_mn, integer=False)
        got = _run(api, torch, A, B, M, N, K, batch, a_mn, b_mn)
        # products of bf16 values are exact in fp32; only the K additions round (<= K * 2^-24 relative to sum |ab|)
        bound = K * 2.0 ** -23 * (K ** 0.5) * 4.0 + 1e-6
        assert (got.double() - ref).abs().max().item() <= bound * 8, (M, N, K, batch)


def test_bgemm_epilogues_and_shared_operand():
    import torch
    from paper_1905_10395_b200 import api
    gen = torch.Generator(device="cuda").manual_seed(7)
    M, N, K, batch = 256, 200, 136, 3
    A, B, ref = _operands(torch, gen, M, N, K, batch, 0, 0, integer=True, share_a=True)
    bias = torch.randint(-3, 4, (batch, N), generator=gen, device="cuda").float()
    got = _run(api, torch, A, B, M, N, K, batch, 0, 0, epilogue=1, bias=bias, share_a=True)
    want = torch.relu(ref + bias[:, None, :].double()).to(torch.bfloat16)
    assert torch.equal(got, want)
    mask = torch.randint(-1, 2, (batch, M, N), generator=gen, device="cuda").to(torch.bfloat16)
    got = _run(api, torch, A, B, M, N, K, batch, 0, 0, epilogue=2, mask=mask, share_a=True)
    want = torch.where(mask.double() > 0, ref, torch.zeros_like(ref)).to(torch.bfloat16)
    assert torch.equal(got, want)
    got = _run(api, torch, A, B, M, N, K, batch, 0, 0, epilogue=3, share_a=True)
    assert torch.equal(got, ref.to(torch.bfloat16))


@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 1)])
def test_bgemm_wide_tiles_on_large_products(a_mn, b_mn):
    """Products with enough tiles use 256-wide tiles (bf16 outputs only): ragged M, N, K, every epilogue."""
    import torch
    from paper_1905_10395_b200 import api
    gen = torch.Generator(device="cuda").manual_seed(31 + 2 * a_mn + b_mn)
    M, N, K, batch = 1000, 1096, 200, 12                      # 8 x 5 x 12 = 480 wide tiles
    A, B, ref = _operands(torch, gen, M, N, K, batch, a_mn, b_mn, integer=True)
    got = _run(api, torch, A, B, M, N, K, batch, a_mn, b_mn, epilogue=3)
    assert torch.equal(got, ref.to(torch.bfloat16))
    bias = torch.randint(-3, 4, (batch, N), generator=gen, device="cuda").float()
    got = _run(api, torch, A, B, M, N, K, batch, a_mn, b_mn, epilogue=1, bias=bias)
    assert torch.equal(got, torch.relu(ref + bias[:, None, :].double()).to(torch.bfloat16))
    mask = torch.randint(-1, 2, (batch, M, N), generator=gen, device="cuda").to(torch.bfloat16)
    got = _run(api, torch, A, B, M, N, K, batch, a_mn, b_mn, epilogue=2, mask=mask)
    assert torch.equal(got, torch.where(mask.double() > 0, ref, torch.zeros_like(ref)).to(torch.bfloat16))


@pytest.mark.parametrize("M,N,K,batch,share_a", [(1024, 1024, 784, 12, False), (512, 768, 1024, 40, True),
                                                 (1000, 1096, 200, 12, False), (300, 264, 72, 80, False)])
def test_bgemm_cta_pair_tiles(M, N, K, batch, share_a):
    """K-major products with bf16 output and at least two rounds of 256 x 256 tiles run on CTA pairs
    (tcgen05 cta_group::2: each CTA of a pair loads half of both operands).  Exact against fp64 on integer
    operands, with full and ragged tiles, a shared A operand (the held-out batch) and both epilogues."""
    import torch
    from paper_1905_10395_b200 import api
    gen = torch.Generator(device="cuda").manual_seed(500 + M + N)
    A, B, ref = _operands(torch, gen, M, N, K, batch, 0, 0, integer=True, share_a=share_a)
    got = _run(api, torch, A, B, M, N, K, batch, 0, 0, epilogue=3, share_a=share_a)
    assert torch.equal(got, ref.to(torch.bfloat16))
    bias = torch.randint(-3, 4, (batch, N), generator=gen, device="cuda").float()
    got = _run(api, torch, A, B, M, N, K, batch, 0, 0, epilogue=1, bias=bias, share_a=share_a)
    assert torch.equal(got, torch.relu(ref + bias[:, None, :].double()).to(torch.bfloat16))
    assert api.lsgd_bgemm_check_device() == 0
