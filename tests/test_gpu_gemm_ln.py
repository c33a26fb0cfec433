"""GPU parity of the ViT-block building blocks (tcgen05 GEMM epilogues, LayerNorm) against the
CPU oracle's plain loops."""
import numpy as np
import pytest
import torch

import oracle
import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2601_12150_b200 as spv
    c = spv.Context(0)
    yield c
    c.close()


def _bf16(dev, a):
    return torch.from_numpy(a).to(dev).to(torch.bfloat16)


def _check(got, ref, max_abs=2e-2, rel_l2=5e-3):
    err = got.astype(np.float64) - ref.astype(np.float64)
    # bf16 output: 2e-2 for the arithmetic plus half a bf16 ulp of the value for the rounding to the output format
    half_ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref.astype(np.float64)), 2.0 ** -126))) - 8)
    assert (np.abs(err) <= max_abs + half_ulp).all(), np.abs(err).max()
    assert np.linalg.norm(err) / max(np.linalg.norm(ref), 1e-30) <= rel_l2


# M <= 256 runs on single CTAs with 128-row tiles, M > 256 on CTA pairs with 256-row tiles.  (257, ...)
# and (385, ...): the odd CTA's half of the last tile lies wholly past M; (256, ...): the largest
# single-CTA problem; (640, 136, ...): a column tile of which the odd CTA's rows of W lie past N;
# (20000, 1288, ...): more tiles than CTA pairs, ragged in M and N, several passes over the ring.
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (300, 512, 192), (1000, 264, 328), (77, 64, 1024),
                                   (4097, 1024, 1024), (257, 256, 128), (385, 512, 64), (256, 512, 200),
                                   (640, 136, 72), (20000, 1288, 456)])
def test_gemm_fp32_residual_epilogue(ctx, M, N, K):
    """resid += scale * (A W^T + bias): fp32 output, so any mis-addressed tile or k-slice shows."""
    import paper_2601_12150_b200 as spv
    rng = np.random.default_rng(M + N + K)
    a = synth.round_bf16(rng.standard_normal((M, K), dtype=np.float32))
    w = synth.round_bf16(rng.standard_normal((N, K), dtype=np.float32) * 0.05)
    bias = rng.standard_normal(N).astype(np.float32)
    scale = rng.standard_normal(N).astype(np.float32)
    resid = rng.standard_normal((M, N)).astype(np.float32)
    dev = ctx.device
    out = torch.from_numpy(resid.copy()).to(dev)
    ctx.gemm_bf16(_bf16(dev, a), _bf16(dev, w), out, spv.EPI_BIAS_SCALE_RESID,
                  bias=torch.from_numpy(bias).to(dev), scale=torch.from_numpy(scale).to(dev))
    ctx.check()
    ref = resid + scale[None] * oracle.linear(a, w, bias)
    assert np.abs(out.cpu().numpy() - ref).max() < 2e-4


@pytest.mark.parametrize("M", [389, 200])          # CTA pairs / single CTAs
@pytest.mark.parametrize("epi", ["bias", "gelu", "silu", "mul", "addrow"])
def test_gemm_epilogues(ctx, epi, M):
    import paper_2601_12150_b200 as spv
    N, K = 520, 136
    rng = np.random.default_rng(5)
    a = synth.round_bf16(rng.standard_normal((M, K), dtype=np.float32))
    w = synth.round_bf16(rng.standard_normal((N, K), dtype=np.float32) * 0.1)
    bias = rng.standard_normal(N).astype(np.float32)
    dev = ctx.device
    lin = oracle.linear(a, w, bias)
    A, W, Bv = _bf16(dev, a), _bf16(dev, w), torch.from_numpy(bias).to(dev)
    if epi == "addrow":
        rpi = 100
        add = rng.standard_normal((rpi, N)).astype(np.float32)
        out = torch.zeros((M, N), dtype=torch.float32, device=dev)
        ctx.gemm_bf16(A, W, out, spv.EPI_BIAS_ADDROW, bias=Bv, addrow=torch.from_numpy(add).to(dev),
                      rows_per_image=rpi)
        ctx.check()
        ref = lin + add[np.arange(M) % rpi]
        assert np.abs(out.cpu().numpy() - ref).max() < 2e-4
        return
    out = torch.zeros((M, N), dtype=torch.bfloat16, device=dev)
    if epi == "bias":
        ctx.gemm_bf16(A, W, out, spv.EPI_BIAS, bias=Bv)
        ref = lin
    elif epi == "gelu":
        ctx.gemm_bf16(A, W, out, spv.EPI_BIAS_GELU, bias=Bv)
        ref = np.vectorize(oracle.gelu)(lin).astype(np.float32)
    elif epi == "silu":
        ctx.gemm_bf16(A, W, out, spv.EPI_BIAS_SILU, bias=Bv)
        ref = np.vectorize(oracle.silu)(lin).astype(np.float32)
    else:
        aux = synth.round_bf16(rng.standard_normal((M, N), dtype=np.float32))
        ctx.gemm_bf16(A, W, out, spv.EPI_BIAS_MUL, bias=Bv, aux=_bf16(dev, aux))
        ref = lin * aux
    ctx.check()
    _check(out.float().cpu().numpy(), ref)


# (4097, 1024), (5000, 1536), (2600, 2304): more rows than the persistent grid has warps, so warps
# walk several rows with the next row's loads in flight, and the last pass is ragged
@pytest.mark.parametrize("rows,dim", [(5, 64), (4097, 1024), (1000, 1536), (33, 2304), (5000, 1536), (2600, 2304),
                                      (9001, 512)])
def test_layernorm(ctx, rows, dim):
    rng = np.random.default_rng(rows)
    x = (rng.standard_normal((rows, dim)) * 3 + 1.5).astype(np.float32)
    g = (1 + 0.1 * rng.standard_normal(dim)).astype(np.float32)
    b = (0.1 * rng.standard_normal(dim)).astype(np.float32)
    dev = ctx.device
    y = ctx.layernorm(torch.from_numpy(x).to(dev), torch.from_numpy(g).to(dev), torch.from_numpy(b).to(dev))
    ctx.check()
    ref = oracle.layernorm(x, g, b, 1e-6)
    _check(y.float().cpu().numpy(), ref)
    # scattered output rows
    perm = torch.randperm(rows, device=dev).to(torch.int32)
    y2 = ctx.layernorm(torch.from_numpy(x).to(dev), torch.from_numpy(g).to(dev), torch.from_numpy(b).to(dev),
                       out_row=perm)
    assert torch.equal(y2[perm.long()], y)


@pytest.mark.parametrize("seed", range(8))
def test_gemm_random_shapes(ctx, seed):
    """Seeded random M (single CTAs and CTA pairs), N and K (multiples of 8, ragged against the 256 x 256 x 64
    tiling) with the fp32 residual epilogue, where every mis-addressed tile, k-slice or bias column shows."""
    import paper_2601_12150_b200 as spv
    rng = np.random.default_rng(300 + seed)
    M = int(rng.choice([rng.integers(1, 257), rng.integers(257, 1500), rng.integers(1500, 6000)]))
    N = 8 * int(rng.integers(1, 140))
    K = 8 * int(rng.integers(1, 80))
    a = synth.round_bf16(rng.standard_normal((M, K), dtype=np.float32))
    w = synth.round_bf16(rng.standard_normal((N, K), dtype=np.float32) * 0.05)
    bias = rng.standard_normal(N).astype(np.float32)
    scale = rng.standard_normal(N).astype(np.float32)
    resid = rng.standard_normal((M, N)).astype(np.float32)
    dev = ctx.device
    out = torch.from_numpy(resid.copy()).to(dev)
    ctx.gemm_bf16(_bf16(dev, a), _bf16(dev, w), out, spv.EPI_BIAS_SCALE_RESID,
                  bias=torch.from_numpy(bias).to(dev), scale=torch.from_numpy(scale).to(dev))
    ctx.check()
    ref = resid + scale[None] * oracle.linear(a, w, bias)
    assert np.abs(out.cpu().numpy() - ref).max() < 2e-4, (M, N, K)
    out2 = torch.zeros((M, N), dtype=torch.bfloat16, device=dev)
    ctx.gemm_bf16(_bf16(dev, a), _bf16(dev, w), out2, spv.EPI_BIAS_GELU, bias=torch.from_numpy(bias).to(dev))
    ctx.check()
    _check(out2.float().cpu().numpy(), np.vectorize(oracle.gelu)(oracle.linear(a, w, bias)).astype(np.float32))
