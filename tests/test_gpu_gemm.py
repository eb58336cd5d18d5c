"""The GEMM kernels on their own, through the C ABI's test hook, against a float64 matmul."""
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2505_19201_b200 import api, configs, synth
    p = configs.scaled("llava7b", n_layers=1, vocab=1024, n_visual=64, k_visual=16, n_prompt=32, decode_steps=2)
    tw, dw = synth.target_weights(p, 0, "cuda:0"), synth.draft_weights(p, 0, "cuda:0")
    c = api.Context(api.make_config(p), tw, dw, "cuda:0")
    yield c
    c.close()


SHAPES = [  # rows, N, K : several tiles, ragged tails, one k-panel, many CTAs per tile; interleaved
    # (<= 64 rows), two-plane (65..128 rows) and chunked (> 128 rows) activation layouts
    (61, 12288, 4096), (61, 4096, 4096), (61, 22016, 4096), (61, 4096, 11008), (1, 32000, 4096),
    (8, 1024, 4096), (128, 4096, 4096), (17, 136, 64), (16, 128, 128), (3, 8, 64), (81, 3840, 3840), (100, 520, 704),
    (64, 264, 192), (65, 256, 128), (244, 4096, 4096),
]


@pytest.mark.parametrize("rows,N,K", SHAPES)
@pytest.mark.parametrize("split", [1, 0])
def test_gemm_matches_float64(ctx, rows, N, K, split):
    if split == 0 and rows > 128:
        pytest.skip("single-row inputs take at most 128 rows per call")
    g = torch.Generator(device="cuda").manual_seed(rows * 7 + N + K)
    W = (torch.randn(N, K, device="cuda", generator=g) * 0.02).to(torch.bfloat16)
    X = torch.randn(rows, K, device="cuda", generator=g)
    tc0, _ = ctx.dream_gemm_counts()
    out = ctx.dream_debug_gemm(W, X, split)
    ctx.dream_poll()
    tc1, _ = ctx.dream_gemm_counts()
    assert tc1 >= tc0 + 1, "the tensor-core kernel did not take this shape"
    Xr = X.double() if split else X.to(torch.bfloat16).double()
    ref = Xr @ W.double().t()
    err = float((out.double() - ref).abs().max())
    scale = float(ref.abs().max())
    assert err <= (2e-5 if split else 1e-5) * scale + 1e-6, f"max err {err:.3e} vs scale {scale:.3e}"


def test_back_to_back_launches_share_the_output_buffer(ctx):
    """Two GEMMs in a row on the same stream: the second overwrites the first one's output only
    after the first one's consumer has read it (dependent launches)."""
    g = torch.Generator(device="cuda").manual_seed(5)
    W1 = (torch.randn(4096, 4096, device="cuda", generator=g) * 0.02).to(torch.bfloat16)
    W2 = (torch.randn(1024, 4096, device="cuda", generator=g) * 0.02).to(torch.bfloat16)
    X = torch.randn(61, 4096, device="cuda", generator=g)
    outs = [(ctx.dream_debug_gemm(W1, X, 1), W1) if i % 2 == 0 else (ctx.dream_debug_gemm(W2, X, 1), W2) for i in range(6)]
    ctx.dream_poll()
    for out, W in outs:
        ref = X.double() @ W.double().t()
        assert float((out.double() - ref).abs().max()) <= 2e-5 * float(ref.abs().max()) + 1e-6
