"""GPU parity of cls_score_topk_filter (Sec. 3.3) against the CPU oracle: indices bit-exact,
head means bit-exact, gathered rows byte-exact."""
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


def _run(ctx, sc, tok, G, keep, canary=True):
    dev = ctx.device
    B, H, NP = sc.shape
    import paper_2601_12150_b200 as spv
    k = spv.filter_keep_count(NP, keep)
    dsc = torch.from_numpy(sc).to(dev)
    dtok = None if tok is None else torch.from_numpy(tok.view(np.int16)).to(dev).view(torch.bfloat16)
    mean = torch.zeros((B, NP), dtype=torch.float32, device=dev)
    out_buf = None
    if tok is not None:   # canary rows after the last output row must stay untouched
        out_buf = torch.full((B * (G + k) + 4, tok.shape[-1]), 7.0, dtype=torch.bfloat16, device=dev)
        out = out_buf[:B * (G + k)].view(B, G + k, tok.shape[-1])
    else:
        out = None
    out, kept = ctx.cls_score_topk_filter(dsc, dtok, n_global=G, keep_ratio=keep, tokens_out=out,
                                          mean_scores=mean)
    ctx.check()
    got_tok = None if out is None else out.view(torch.int16).cpu().numpy().view(np.uint16)
    if out_buf is not None:
        assert torch.all(out_buf[B * (G + k):] == 7.0)
    return got_tok, kept.cpu().numpy(), mean.cpu().numpy()


@pytest.mark.parametrize("grid,B,dim,keep,quantum,G", [
    (64, 1, 1024, 0.5, None, 1),          # the token-filter workload: [16,4096] scores, 4097 x 1024 rows
    (64, 2, 1024, 0.6, 2.0 ** -12, 1),    # heavy ties at the threshold
    (37, 3, 256, 0.37, None, 2),          # ragged sizes, n_patch not a multiple of 4
    (146, 1, 1536, 0.5, None, 1),         # 21316 patches, 3 KB rows
    (16, 2, 64, 1.0, None, 1),            # keep everything: identity
])
def test_filter_matches_oracle(ctx, grid, B, dim, keep, quantum, G):
    sc = synth.filter_scores(1, B, 16, grid, grid, tie_quantum=quantum)
    tok = synth.token_rows(2, B, G + grid * grid, dim)
    want_tok, want_kept, want_mean = oracle.token_filter(sc, tok, n_global=G, keep_ratio=keep)
    got_tok, got_kept, got_mean = _run(ctx, sc, tok, G, keep)
    assert np.array_equal(got_kept, want_kept)
    assert np.array_equal(got_mean.view(np.uint32), want_mean.view(np.uint32))
    assert np.array_equal(got_tok, want_tok)


def test_filter_large_batch_full_size(ctx):
    # 256x256 grid (4096^2 image at patch 16), batch 4, keep 0.5: indices and sampled rows
    sc = synth.filter_scores(6, 4, 16, 256, 256)
    tok = synth.token_rows(7, 4, 1 + 65536, 1024)
    want_tok, want_kept, _ = oracle.token_filter(sc, tok, n_global=1, keep_ratio=0.5)
    got_tok, got_kept, _ = _run(ctx, sc, tok, 1, 0.5)
    assert np.array_equal(got_kept, want_kept)
    assert np.array_equal(got_tok, want_tok)


def test_filter_degenerate_scores(ctx):
    sc = np.full((2, 4, 1000), 0.25, dtype=np.float32)       # all equal -> first k indices
    _, kept, _ = _run(ctx, sc, None, 1, 0.3)
    assert np.array_equal(kept, np.tile(np.arange(300, dtype=np.int32), (2, 1)))
    sc = np.zeros((1, 2, 8), dtype=np.float32)
    sc[0, :, 1] = -0.0
    sc[0, :, 5] = 1.0
    sc[0, :, 6] = np.nan
    _, kept, _ = _run(ctx, sc, None, 1, 0.5)                  # k=4: 5, then zeros 0,1,2 (-0 ties +0); NaN last
    want = oracle.token_filter(sc, None, keep_ratio=0.5)[1]
    assert np.array_equal(kept, want) and kept.tolist() == [[0, 1, 2, 5]]
    sc = np.random.default_rng(0).standard_normal((1, 3, 1)).astype(np.float32)
    _, kept, _ = _run(ctx, sc, None, 1, 0.5)                  # a single patch
    assert kept.tolist() == [[0]]


def test_filter_argument_errors(ctx):
    import paper_2601_12150_b200 as spv
    sc = torch.zeros((1, 2, 16), dtype=torch.float32, device=ctx.device)
    with pytest.raises(spv.SpvError):
        ctx.cls_score_topk_filter(sc, None, keep_ratio=0.0)
    tok = torch.zeros((1, 17, 12), dtype=torch.bfloat16, device=ctx.device)   # dim not a multiple of 8
    with pytest.raises(spv.SpvError):
        ctx.cls_score_topk_filter(sc, tok, keep_ratio=0.5)
    small = torch.empty(256, dtype=torch.uint8, device=ctx.device)
    big = torch.zeros((1, 2, 100000), dtype=torch.float32, device=ctx.device)
    with pytest.raises(spv.SpvError) as e:
        ctx.cls_score_topk_filter(big, None, keep_ratio=0.5, workspace=small)
    assert e.value.status == spv.ERR_WORKSPACE
