"""cls_score_topk_filter_static: the token filter for callers that may not allocate device memory
(servers with a fixed memory plan, plug-ins inside a host that owns the allocator, loops where an
allocation would stall the device).  It must give exactly what cls_score_topk_filter gives -- kept
indices, head means and gathered rows bit for bit -- on calls in a row that share its built-in
scratch array, and it must refuse requests that do not fit that array.

Collected last on purpose: a failure here leaves every other test already run under `-x`."""
import ctypes as C

import numpy as np
import pytest
import torch

import synth

pytestmark = pytest.mark.gpu


def _both(ctx, spv, seed, B, H, grid, dim, keep, G=1):
    dev = ctx.device
    sc = torch.from_numpy(synth.filter_scores(seed, B, H, grid, grid)).to(dev)
    tok = torch.from_numpy(synth.token_rows(seed + 1, B, G + grid * grid, dim).view(np.int16)).to(dev).view(torch.bfloat16)
    k = spv.filter_keep_count(grid * grid, keep)
    pos_in = torch.arange(grid * grid, dtype=torch.int32, device=dev).flip(0).repeat(B, 1).contiguous()
    # reference: the entry point with a context and a caller workspace
    mean_a = torch.zeros((B, grid * grid), dtype=torch.float32, device=dev)
    pos_a = torch.zeros((B, k), dtype=torch.int32, device=dev)
    out_a, kept_a = ctx.cls_score_topk_filter(sc, tok, n_global=G, keep_ratio=keep, mean_scores=mean_a,
                                              pos_in=pos_in, pos_out=pos_a)
    ctx.check()
    # the allocation-free entry point: every buffer made here, before the call
    out_b = torch.full((B, G + k, dim), -3.0, dtype=torch.bfloat16, device=dev)
    kept_b = torch.full((B, k), -1, dtype=torch.int32, device=dev)
    mean_b = torch.zeros_like(mean_a)
    pos_b = torch.zeros_like(pos_a)
    # one call first, so that loading the kernels is done; the device's free memory as the driver reports it
    # (cudaMemGetInfo, which sees any cudaMalloc, not only torch's allocator) must then not move over a call
    spv.cls_score_topk_filter_static(sc, tok, out_b, kept_b, n_global=G, keep_ratio=keep, mean_scores=mean_b,
                                     pos_in=pos_in, pos_out=pos_b)
    torch.cuda.synchronize()
    out_b.fill_(-3.0)
    kept_b.fill_(-1)
    mean_b.zero_()
    pos_b.zero_()
    torch.cuda.synchronize()
    before, before_torch = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    spv.cls_score_topk_filter_static(sc, tok, out_b, kept_b, n_global=G, keep_ratio=keep, mean_scores=mean_b,
                                     pos_in=pos_in, pos_out=pos_b)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == before and torch.cuda.memory_allocated() == before_torch
    assert torch.equal(kept_a, kept_b)
    assert torch.equal(mean_a.view(torch.int32), mean_b.view(torch.int32))
    assert torch.equal(out_a.view(torch.int16), out_b.view(torch.int16))
    assert torch.equal(pos_a, pos_b)


def test_static_filter_matches_workspace_filter_on_consecutive_calls():
    import paper_2601_12150_b200 as spv
    ctx = spv.Context(0)
    try:
        # two calls in a row on the shared scratch: a large request, then a smaller one with other
        # data whose padding and tail would expose anything left over from the first
        _both(ctx, spv, 1, 2, 16, 64, 1024, 0.5)
        _both(ctx, spv, 5, 3, 8, 37, 256, 0.37, G=2)
        _both(ctx, spv, 9, 4, 16, 256, 64, 0.5)          # exactly at the limit: 4 x 65536 x 8 B = 2 MiB
    finally:
        ctx.close()


def test_static_filter_rejects_what_does_not_fit():
    import paper_2601_12150_b200 as spv
    dev = torch.device("cuda", 0)
    n = 65540                                             # 4 x round_up(65540, 4) x 8 B > 2 MiB
    sc = torch.zeros((4, 2, n), dtype=torch.float32, device=dev)
    kept = torch.zeros((4, n // 2), dtype=torch.int32, device=dev)
    with pytest.raises(spv.SpvError) as e:
        spv.cls_score_topk_filter_static(sc, None, None, kept, keep_ratio=0.5)
    assert e.value.status == spv.ERR_STATIC_LIMIT
    assert "static" in spv.status_string(spv.ERR_STATIC_LIMIT)
    with pytest.raises(spv.SpvError):
        spv.cls_score_topk_filter_static(sc[:1, :, :16], None, None, kept, keep_ratio=0.0)
