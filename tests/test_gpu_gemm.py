"""The projection GEMM kernels against a plain fp64 matrix product (numpy) on the same bf16 inputs."""
import numpy as np
import pytest
import torch

from paper_2511_18793_b200 import synth
from gpu_helpers import Case

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    w = synth.scaled(synth.WORKLOADS["small"], n_items=10_000, n_layers=1, batch=2, n_hist=2)
    return Case(w)


def _ref(A, W):
    return A.double().cpu().numpy() @ W.double().cpu().numpy().T


@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (200, 256, 512), (1920, 1536, 512), (77, 768, 2048), (640, 512, 1024),
                                    (1, 128, 64), (129, 128, 4864),
                                    # large enough for the CTA-pair kernel (256 x 256 tiles), ragged in M and in N
                                    (5000, 2304, 896), (18000, 1152, 512), (4100, 512, 2048)])
@pytest.mark.parametrize("path", [1, 2, 3])
def test_gemm_epilogues(ctx, M, N, K, path):
    g = torch.Generator(device="cuda"); g.manual_seed(M * 7 + N * 3 + K)
    A = (torch.randn(M, K, generator=g, device="cuda") * 0.5).bfloat16()
    W = (torch.randn(N, K, generator=g, device="cuda") * 0.05).bfloat16()
    ref = _ref(A, W)
    scale = np.abs(ref).max()
    out = torch.empty(M, N, dtype=torch.float32, device="cuda")
    ctx.eng.gemm(A, W, out, epilogue=1, path=path)
    assert np.abs(out.cpu().numpy() - ref).max() < 2e-5 * scale * np.sqrt(K / 64) + 1e-6      # fp32 accumulation only
    outb = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    ctx.eng.gemm(A, W, outb, epilogue=0, path=path)
    assert np.abs(outb.float().cpu().numpy() - ref).max() < scale * 2 ** -8
    res = torch.randn(M, N, generator=g, device="cuda")
    acc = res.clone()
    ctx.eng.gemm(A, W, acc, epilogue=2, path=path)
    assert np.abs(acc.cpu().numpy() - (res.double().cpu().numpy() + ref)).max() < 2e-5 * scale * np.sqrt(K / 64) + 1e-5
    bias = torch.randn(N, generator=g, device="cuda")
    th = torch.empty(M, N, dtype=torch.float32, device="cuda")
    ctx.eng.gemm(A, W, th, epilogue=3, bias=bias, path=path)
    assert np.abs(th.cpu().numpy() - np.tanh(ref + bias.double().cpu().numpy())).max() < 1e-4
    ctx.eng.sync()


def test_gemm_tc_rejects_uncovered_shapes(ctx):
    A = torch.zeros(8, 48, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(128, 48, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(8, 128, dtype=torch.float32, device="cuda")
    with pytest.raises(ctx.binding.NezhaError) as ei:
        ctx.eng.gemm(A, W, out, epilogue=1, path=2)
    assert ei.value.status == 7
    ctx.eng.gemm(A, W, out, epilogue=1, path=0)          # falls back to the CUDA-core kernel
    ctx.eng.sync()


@pytest.mark.parametrize("path", [2, 3])
@pytest.mark.parametrize("N,K", [(512, 2048), (768, 512), (1536, 512), (4096, 512), (896, 4864)])
def test_gemm_rows_do_not_depend_on_the_number_of_rows(ctx, N, K, path):
    """A row of the product must come out with the same bits whatever the launch's row count (which decides the tile
    width, the kernel and the number of waves): the two decode modes run passes of different sizes and must agree exactly."""
    g = torch.Generator(device="cuda"); g.manual_seed(N + K)
    A = (torch.randn(5200, K, generator=g, device="cuda") * 0.5).bfloat16()
    W = (torch.randn(N, K, generator=g, device="cuda") * 0.05).bfloat16()
    full = torch.empty(5200, N, dtype=torch.float32, device="cuda")
    ctx.eng.gemm(A, W, full, epilogue=1, path=path)
    for M in (1, 77, 640, 1920):
        part = torch.empty(M, N, dtype=torch.float32, device="cuda")
        ctx.eng.gemm(A[:M].contiguous(), W, part, epilogue=1, path=path)
        assert torch.equal(part, full[:M]), (N, K, path, M)
    ctx.eng.sync()


@pytest.mark.parametrize("path", [2, 3])
@pytest.mark.parametrize("N,K", [(512, 192), (896, 320), (1024, 576), (256, 960), (64, 192)])
def test_gemm_odd_number_of_k_steps_many_tiles_per_cta(ctx, N, K, path):
    """K / 64 odd and far more output tiles than SMs: every CTA walks several tiles, so the operand ring's slots change
    hands between tiles unless the kernel keeps one waiter per slot.  Against the fp64 product, and twice (bit-equal)."""
    M = 128 * 148 * 3 + 77
    g = torch.Generator(device="cuda"); g.manual_seed(N * 5 + K)
    A = (torch.randn(M, K, generator=g, device="cuda") * 0.5).bfloat16()
    W = (torch.randn(N, K, generator=g, device="cuda") * 0.05).bfloat16()
    ref = _ref(A, W)
    scale = np.abs(ref).max()
    out = torch.empty(M, N, dtype=torch.float32, device="cuda")
    ctx.eng.gemm(A, W, out, epilogue=1, path=path)
    assert np.abs(out.cpu().numpy() - ref).max() < 2e-5 * scale * np.sqrt(K / 64) + 1e-6
    again = torch.empty_like(out)
    ctx.eng.gemm(A, W, again, epilogue=1, path=path)
    assert torch.equal(out, again)
    ctx.eng.sync()


@pytest.mark.parametrize("N,K", [(512, 512), (3072, 2048), (2048, 8192), (2080, 2048), (16384, 2048), (32, 64), (256, 192)])
def test_weight_streaming_gemm(ctx, N, K):
    """The kernel for launches of at most 128 rows (weights as the 128-row MMA operand, K split over CTAs): every epilogue
    against the fp64 product, for row counts in each of its three accumulator widths (32, 64, 128); a row's bits depend neither on the
    number of rows nor on the order in which the CTAs of a tile arrive (run twice)."""
    g = torch.Generator(device="cuda"); g.manual_seed(N * 11 + K)
    A64 = (torch.randn(128, K, generator=g, device="cuda") * 0.5).bfloat16()
    W = (torch.randn(N, K, generator=g, device="cuda") * 0.05).bfloat16()
    bias = torch.randn(N, generator=g, device="cuda")
    res64 = torch.randn(128, N, generator=g, device="cuda")
    ref64 = _ref(A64, W)                                    # (also a device synchronisation: W is at rest from here on)
    scale = np.abs(ref64).max()
    full = torch.empty(128, N, dtype=torch.float32, device="cuda")
    ctx.eng.gemm(A64, W, full, epilogue=1, path=4)
    for M in (1, 7, 20, 32, 33, 50, 64, 65, 97, 128):
        A, ref = A64[:M].contiguous(), ref64[:M]
        out = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        ctx.eng.gemm(A, W, out, epilogue=1, path=4)
        assert np.abs(out.cpu().numpy() - ref).max() < 2e-5 * scale * np.sqrt(K / 64) + 1e-6
        assert torch.equal(out, full[:M]), (N, K, M)
        again = torch.empty_like(out)
        ctx.eng.gemm(A, W, again, epilogue=1, path=4)
        assert torch.equal(out, again)
        outb = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
        ctx.eng.gemm(A, W, outb, epilogue=0, path=4)
        assert np.abs(outb.float().cpu().numpy() - ref).max() < scale * 2 ** -8
        acc = res64[:M].clone()
        ctx.eng.gemm(A, W, acc, epilogue=2, path=4)
        assert np.abs(acc.cpu().numpy() - (res64[:M].double().cpu().numpy() + ref)).max() < 2e-5 * scale * np.sqrt(K / 64) + 1e-5
        th = torch.empty(M, N, dtype=torch.float32, device="cuda")
        ctx.eng.gemm(A, W, th, epilogue=3, bias=bias, path=4)
        assert np.abs(th.cpu().numpy() - np.tanh(ref + bias.double().cpu().numpy())).max() < 1e-4
    ctx.eng.sync()


def test_weight_streaming_gemm_takes_at_most_128_rows(ctx):
    A = torch.zeros(129, 64, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(129, 128, dtype=torch.float32, device="cuda")
    with pytest.raises(ctx.binding.NezhaError) as ei:
        ctx.eng.gemm(A, W, out, epilogue=1, path=4)
    assert ei.value.status == 7
