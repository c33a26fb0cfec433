"""GPU parity of vit_forward (Sec. 3 / Sec. 4.1 backbone with the sparse attention of Sec. 3.2 and
the token filter of Sec. 3.3) against the CPU oracle on the same seeded weights and images.

Tolerance for the bf16 output tokens vs the oracle: max |err| <= 2e-2 and relative L2 <= 5e-3.
The filter decides an integer result from scores that the two sides compute in different
precisions, so the comparison runs twice: free-running (kept sets may differ only in tokens whose
oracle score sits within THRESHOLD_REL of the oracle's threshold score) and teacher-forced (the
oracle is re-run with the GPU's kept indices, then the tensor tolerances apply).

THRESHOLD_REL = 2^-8: the GPU forms the CLS logits from bf16 q and k, i.e. from operands that carry a
relative rounding error of up to half a bf16 ulp, 2^-8; a softmax weight inherits the logit's absolute
error as a relative one.  With trained-looking (peaked) score rows few tokens sit that close to the
threshold; with the nearly uniform rows random weights give on a 146x146 grid (every weight within a few
1e-4 relative of 1/N) the ranking near the threshold is decided below the operands' precision, and the
bound says exactly how far a disagreeing token may be from it."""
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


THRESHOLD_REL = 2.0 ** -8


def _half_ulp_bf16(x):
    """Half a unit in the last place of the bf16 number nearest to x (8 significand bits)."""
    ax = np.maximum(np.abs(np.asarray(x, dtype=np.float64)), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - 8)


def _check(got, ref, max_abs=2e-2, rel_l2=5e-3):
    """max |err| <= 2e-2 and relative L2 <= 5e-3.  The outputs are stored as bf16: the 2e-2 is the budget of
    the arithmetic (the value before it is rounded to the output format), and the rounding itself may add up
    to half a bf16 ulp of the value, which alone passes 2e-2 from |x| = 4 on.  Element bound: 2e-2 + half_ulp."""
    assert np.isfinite(got).all()
    err = got.astype(np.float64) - ref.astype(np.float64)
    bound = max_abs + _half_ulp_bf16(ref)
    worst = np.unravel_index(np.argmax(np.abs(err) / bound), err.shape)
    assert (np.abs(err) <= bound).all(), (worst, float(err[worst]), float(ref[worst]))
    rel = np.linalg.norm(err) / np.linalg.norm(ref)
    assert rel <= rel_l2, rel


def _gpu_forward(ctx, cfg, w, image, gh, gw, forced_keep=None):
    dev = ctx.device
    dw = ctx.make_vit_weights(w)
    fk = None if forced_keep is None else torch.from_numpy(np.ascontiguousarray(forced_keep, dtype=np.int32)).to(dev)
    out, kept = ctx.vit_forward(cfg, dw, torch.from_numpy(image).to(dev), gh, gw, forced_keep=fk)
    ctx.check()
    return out.float().cpu().numpy(), None if kept is None else kept.cpu().numpy()


def _mean_scores_of_oracle(cfg, w, image, gh, gw):
    """Head-averaged CLS scores the oracle ranks on: rerun with keep 1.0 is not needed -- the tap of
    the residual stream cannot give them, so recompute the filter layer's scores from a forward
    truncated at that layer with the filter off and `want_scores`-style attention of its input."""
    c = dict(cfg)
    c["layers"] = cfg["filter_layer"]
    c["filter_layer"] = 0
    tap_l = cfg["filter_layer"] - 1
    x = oracle.vit_forward(c, dict(w, layers=w["layers"][:c["layers"]]), image, gh, gw, tap_layer=tap_l)["tap"]
    lw = w["layers"][tap_l]
    D, H = cfg["dim"], cfg["heads"]
    h = oracle.layernorm(x, lw["ln1_g"], lw["ln1_b"], cfg["ln_eps"])
    qkv = oracle.linear(h, lw["w_qkv"], lw["b_qkv"])
    B, N = x.shape[:2]
    q, k, v = (np.ascontiguousarray(qkv[..., i * D:(i + 1) * D]).reshape(B, N, H, D // H) for i in range(3))
    dense = cfg["attn_mode"] == synth.ATTN_DENSE
    _, sc = oracle.attention(q, k, v, gh, gw, 1 if dense else cfg["block"], max(gh, gw) if dense else cfg["radius"],
                             n_global=cfg["n_global"], want_scores=True)
    return oracle.token_filter(sc, None, n_global=cfg["n_global"], keep_ratio=1.0)[2]


def _stage_counts(cfg, npatch):
    stages = cfg.get("filters") or ([(cfg["filter_layer"], cfg["keep_ratio"])] if cfg.get("filter_layer", 0) > 0 else [])
    out, cur = [], npatch
    for _, ratio in stages:
        cur = int(np.ceil(ratio * cur - 1e-9))
        out.append(cur)
    return out


def _compare(ctx, arch, cfg, gh, gw, B, seed, w=None, image=None, report=None, free_oracle=None):
    """Free-running, then teacher-forced comparison of one configuration (see the module docstring).  With
    several filter stages the threshold rule is applied to the first stage (the later ones rank different
    token sets once a first-stage token differs); every stage's set must be ascending, of the right size and
    inside the stage before, and the teacher-forced tensors must meet the tolerances."""
    P = arch["patch"]
    if w is None:
        w = synth.vit_weights(seed, arch, gh, gw, pos_base=4)
    if image is None:
        image = synth.tissue_batch(seed + 1, B, gh * P, gw * P, background=0.4)
    full = dict(arch, **cfg)
    got, kept = _gpu_forward(ctx, full, w, image, gh, gw)
    ref = free_oracle() if free_oracle else oracle.vit_forward(full, w, image, gh, gw)
    counts = _stage_counts(full, gh * gw)
    def fill_report(ref_out):
        if report is None:
            return
        err = got.astype(np.float64) - ref_out.astype(np.float64)
        report["max_abs_err"] = float(np.abs(err).max())
        report["rel_l2"] = float(np.linalg.norm(err) / np.linalg.norm(ref_out))
        report["max_err_over_bound"] = float((np.abs(err) / (2e-2 + _half_ulp_bf16(ref_out))).max())
        report["elements"] = int(err.size)
        report["elements_over_2e-2"] = int((np.abs(err) > 2e-2).sum())
        report["max_abs_ref"] = float(np.abs(ref_out).max())

    if not counts:
        assert kept is None
        fill_report(ref["out"])
        _check(got, ref["out"])
        return
    okept = ref["kept_all"]
    assert kept.shape == okept.shape == (B, sum(counts))
    off, prev = 0, None
    for c in counts:
        seg = kept[:, off:off + c]
        assert (np.diff(seg, axis=1) > 0).all() and seg.min() >= 0 and seg.max() < gh * gw
        if prev is not None:
            assert all(np.isin(seg[b], prev[b]).all() for b in range(B))
        prev, off = seg, off + c
    agree = np.array_equal(kept, okept)
    if report is not None:
        report["kept_sets_equal"] = bool(agree)
        report["kept_differ"] = int(sum(np.setxor1d(kept[b], okept[b]).size for b in range(B)))
    if not agree:
        k1 = counts[0]
        if not np.array_equal(kept[:, :k1], okept[:, :k1]):
            first = dict(full)
            if full.get("filters"):
                first.pop("filters")
                first["filter_layer"], first["keep_ratio"] = full["filters"][0]
            mean = _mean_scores_of_oracle(first, w, image, gh, gw)
            worst = 0.0
            for b in range(B):
                thr = np.sort(mean[b])[::-1][k1 - 1]
                diff = np.setxor1d(kept[b, :k1], okept[b, :k1])
                if diff.size:
                    worst = max(worst, float((np.abs(mean[b][diff] - thr) / abs(thr)).max()))
            if report is not None:
                report["max_rel_distance_to_threshold_of_differing_tokens"] = worst
            assert worst <= THRESHOLD_REL, worst
        ref = oracle.vit_forward(full, w, image, gh, gw, forced_keep=kept)
    fill_report(ref["out"])
    _check(got, ref["out"])
    # teacher forcing through the library's own forced_keep argument reproduces its free run
    got2, kept2 = _gpu_forward(ctx, full, w, image, gh, gw, forced_keep=kept)
    assert np.array_equal(kept2, kept)
    assert np.array_equal(got2, got)


@pytest.mark.parametrize("gh,gw,block,radius,filter_layer,keep,B,mlp,patch,G", [
    (16, 16, 8, 1, 0, 1.0, 1, synth.MLP_GELU, 4, 1),      # sparse, no filter, exact tiles
    (16, 16, 8, 1, 1, 0.6, 2, synth.MLP_GELU, 4, 1),      # sparse + filter after block 1
    (13, 21, 8, 1, 2, 0.5, 2, synth.MLP_SWIGLU, 2, 1),    # ragged grid, SwiGLU, im2col width 12 (padded)
    (18, 18, 4, 2, 1, 0.37, 1, synth.MLP_GELU, 4, 2),     # 5x5 neighbourhood, two global tokens
    (12, 20, 8, 0, 3, 0.8, 1, synth.MLP_GELU, 4, 1),      # own block only, filter after the last block
])
def test_vit_forward_sparse(ctx, gh, gw, block, radius, filter_layer, keep, B, mlp, patch, G):
    arch = synth.vit_tiny(layers=3, dim=128, heads=2, hidden=256, patch=patch, mlp_kind=mlp,
                          layerscale=1 if mlp == synth.MLP_GELU else 0, n_global=G)
    cfg = dict(attn_mode=synth.ATTN_SPARSE, block=block, radius=radius, filter_layer=filter_layer, keep_ratio=keep)
    _compare(ctx, arch, cfg, gh, gw, B, seed=gh * 31 + gw)


@pytest.mark.parametrize("gh,gw,block,radius,stages,B,mlp,G", [
    (16, 16, 8, 1, [(1, 0.6), (2, 0.5)], 2, synth.MLP_GELU, 1),          # two stages on exact tiles
    (13, 21, 4, 1, [(1, 0.75), (3, 0.4)], 1, synth.MLP_SWIGLU, 1),       # ragged grid, second stage after the last block
    (20, 12, 8, 2, [(1, 0.8), (2, 0.7), (3, 0.5)], 2, synth.MLP_GELU, 2),  # three stages, 5x5 neighbourhood
])
def test_vit_forward_several_filter_stages(ctx, gh, gw, block, radius, stages, B, mlp, G):
    """Sec. 3.3 applied at more than one block: each stage ranks the tokens still present; survivors keep
    their original positions for the neighbourhood rule."""
    arch = synth.vit_tiny(layers=3, dim=128, heads=2, hidden=256, patch=4, mlp_kind=mlp,
                          layerscale=1 if mlp == synth.MLP_GELU else 0, n_global=G)
    cfg = dict(attn_mode=synth.ATTN_SPARSE, block=block, radius=radius, filters=stages)
    _compare(ctx, arch, cfg, gh, gw, B, seed=gh * 17 + gw)


def test_vit_forward_one_stage_list_equals_single_fields(ctx):
    arch = synth.vit_tiny(layers=2, dim=128, heads=2, hidden=256, patch=4)
    gh, gw = 16, 12
    w = synth.vit_weights(3, arch, gh, gw, pos_base=4)
    image = synth.tissue_batch(4, 2, gh * 4, gw * 4)
    base = dict(arch, attn_mode=synth.ATTN_SPARSE, block=8, radius=1)
    a, ka = _gpu_forward(ctx, dict(base, filter_layer=1, keep_ratio=0.55), w, image, gh, gw)
    b, kb = _gpu_forward(ctx, dict(base, filters=[(1, 0.55)]), w, image, gh, gw)
    assert np.array_equal(a, b) and np.array_equal(ka, kb)


@pytest.mark.parametrize("stages,G", [([(1, 0.5)], 1), ([(1, 0.7), (2, 0.45)], 2), ([(1, 0.6)], 5)])
def test_fused_filter_front_end_is_bit_identical(ctx, stages, G):
    """The filter's fused front end (softmax weights of the CLS row, head mean and ranking keys in one kernel,
    no [batch, heads, patches] score tensor) keeps exactly the tokens the two separate kernels keep."""
    arch = synth.vit_tiny(layers=3, dim=128, heads=2, hidden=256, patch=4, n_global=G)
    gh, gw = 21, 19
    w = synth.vit_weights(8, arch, gh, gw, pos_base=4)
    image = synth.tissue_batch(9, 3, gh * 4, gw * 4)
    cfg = dict(arch, attn_mode=synth.ATTN_SPARSE, block=4, radius=1, filters=stages)
    a, ka = _gpu_forward(ctx, cfg, w, image, gh, gw)
    b, kb = _gpu_forward(ctx, dict(cfg, unfused_filter=1), w, image, gh, gw)
    assert np.array_equal(ka, kb)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("G", [5, 9, 16])
def test_vit_forward_register_tokens(ctx, G):
    """CLS plus register tokens as global tokens (all attend everything and are attended by everything; the
    ranking uses token 0's row; global tokens are never pruned)."""
    arch = synth.vit_tiny(layers=2, dim=128, heads=2, hidden=256, patch=4, n_global=G)
    cfg = dict(attn_mode=synth.ATTN_SPARSE, block=8, radius=1, filter_layer=1, keep_ratio=0.5)
    _compare(ctx, arch, cfg, 18, 14, 1, seed=40 + G)


def test_vit_forward_dense_equals_wide_radius(ctx):
    arch = synth.vit_tiny(layers=2, dim=128, heads=2, hidden=256, patch=4)
    gh, gw = 14, 14
    w = synth.vit_weights(5, arch, gh, gw, pos_base=4)
    image = synth.tissue_batch(6, 1, gh * 4, gw * 4)
    dense = dict(arch, attn_mode=synth.ATTN_DENSE, block=8, radius=1)
    wide = dict(arch, attn_mode=synth.ATTN_SPARSE, block=8, radius=1)     # 2x2 blocks: radius 1 covers the grid
    a, _ = _gpu_forward(ctx, dense, w, image, gh, gw)
    b, _ = _gpu_forward(ctx, wide, w, image, gh, gw)
    assert np.array_equal(a, b)
    _check(a, oracle.vit_forward(dense, w, image, gh, gw)["out"])


def test_vit_forward_wide_model_layer_growth(ctx):
    """d = 1024, 16 heads, hidden 4096 (the ViT-L/16 block shapes) on a 16x16 grid, 4 layers with the
    filter after block 2: the full-width GEMM shapes of the forward against the oracle."""
    arch = dict(synth.vit_l16(), layers=4)
    cfg = dict(attn_mode=synth.ATTN_SPARSE, block=8, radius=1, filter_layer=2, keep_ratio=0.6)
    _compare(ctx, arch, cfg, 16, 16, 1, seed=2)


def test_vit_forward_g14_style_block_shapes(ctx):
    """d = 1536, 24 heads, SwiGLU hidden 4096, patch 14 (im2col width 588, padded to 592), no
    LayerScale: the ViT-g/14-style block shapes on a ragged 18x11 grid, 5x5 neighbourhood, 2 layers
    with the filter after block 1."""
    arch = dict(synth.vit_g14(), layers=2)
    cfg = dict(attn_mode=synth.ATTN_SPARSE, block=8, radius=2, filter_layer=1, keep_ratio=0.5)
    _compare(ctx, arch, cfg, 18, 11, 1, seed=4)


def test_vit_forward_argument_errors(ctx):
    import paper_2601_12150_b200 as spv
    arch = synth.vit_tiny(layers=1, dim=128, heads=2, hidden=256, patch=4)
    w = synth.vit_weights(1, arch, 8, 8, pos_base=4)
    dw = ctx.make_vit_weights(w)
    img = torch.zeros((1, 3, 32, 32), device=ctx.device)
    bad = dict(arch, attn_mode=synth.ATTN_SPARSE, block=8, radius=1, heads=4)          # head_dim 32
    with pytest.raises(spv.SpvError) as e:
        ctx.vit_forward(bad, dw, img, 8, 8)
    assert e.value.status == spv.ERR_UNSUPPORTED
    ok = dict(arch, attn_mode=synth.ATTN_SPARSE, block=8, radius=1)
    small = torch.empty(1024, dtype=torch.uint8, device=ctx.device)
    with pytest.raises(spv.SpvError) as e:
        ctx.vit_forward(ok, dw, img, 8, 8, workspace=small)
    assert e.value.status == spv.ERR_WORKSPACE
    with pytest.raises(spv.SpvError):
        ctx.vit_forward(dict(ok, filter_layer=2, keep_ratio=0.5), dw, img, 8, 8)                       # beyond the last block


def test_index_inputs_are_checked_on_the_device(ctx):
    """forced_keep with a duplicate, an unsorted pair or an entry outside the first stage's set, and an
    unsorted patch_pos: the kernels that read them latch the violation, check() reports INVALID_ARG, and the
    context keeps working."""
    import paper_2601_12150_b200 as spv
    arch = synth.vit_tiny(layers=2, dim=128, heads=2, hidden=256, patch=4)
    gh, gw = 8, 8
    w = synth.vit_weights(1, arch, gh, gw, pos_base=4)
    dw = ctx.make_vit_weights(w)
    img = torch.from_numpy(synth.tissue_batch(2, 1, gh * 4, gw * 4)).to(ctx.device)
    cfg = dict(arch, attn_mode=synth.ATTN_SPARSE, block=4, radius=1, filter_layer=1, keep_ratio=0.5)
    good = np.arange(0, 64, 2, dtype=np.int32)[None]
    out_ok, _ = ctx.vit_forward(cfg, dw, img, gh, gw, forced_keep=torch.from_numpy(good).to(ctx.device))
    ctx.check()
    ref = out_ok.clone()
    for bad in (np.concatenate([good[0, :5], good[0, 4:31]])[None],          # duplicate
                np.concatenate([good[0, 1:2], good[0, 0:1], good[0, 2:]])[None],   # unsorted
                np.concatenate([good[0, :31], [64]])[None].astype(np.int32)):       # outside the grid
        ctx.vit_forward(cfg, dw, img, gh, gw, forced_keep=torch.from_numpy(np.ascontiguousarray(bad, dtype=np.int32)).to(ctx.device))
        with pytest.raises(spv.SpvError) as e:
            ctx.check()
        assert e.value.status == spv.ERR_INVALID_ARG
    two = dict(cfg, filters=[(1, 0.5), (2, 0.5)])
    two.pop("filter_layer"); two.pop("keep_ratio")
    second_bad = np.concatenate([good[0], np.arange(1, 33, 2)]).astype(np.int32)[None]   # stage 2 not inside stage 1
    ctx.vit_forward(two, dw, img, gh, gw, forced_keep=torch.from_numpy(second_bad).to(ctx.device))
    with pytest.raises(spv.SpvError) as e:
        ctx.check()
    assert e.value.status == spv.ERR_INVALID_ARG
    # unsorted patch_pos of the attention entry point
    q = torch.randn((1, 1 + 16, 2, 64), device=ctx.device).to(torch.bfloat16)
    pos = torch.tensor([[0, 1, 2, 3, 8, 9, 10, 11, 5, 4, 6, 7, 12, 13, 14, 15]], dtype=torch.int32, device=ctx.device)
    ctx.spatial_block_attention(q, q, q, 4, 4, 2, 1, patch_pos=pos)
    with pytest.raises(spv.SpvError) as e:
        ctx.check()
    assert e.value.status == spv.ERR_INVALID_ARG
    # the context is still usable and gives the same result as before
    out2, _ = ctx.vit_forward(cfg, dw, img, gh, gw, forced_keep=torch.from_numpy(good).to(ctx.device))
    ctx.check()
    assert torch.equal(out2, ref)


def test_bounded_wait_expires_and_context_survives(ctx):
    """A wait nobody satisfies gives up after its limit: the kernel returns, check() reports the timeout with
    the site code, and the next call works."""
    import paper_2601_12150_b200 as spv
    ctx.selftest_wait(limit_ns=200000)
    with pytest.raises(spv.SpvError) as e:
        ctx.check()
    assert e.value.status == spv.ERR_TIMEOUT
    assert spv.lib().spv_last_wait_site(ctx.handle) == 0x5E1F
    ctx.check()                                   # the latch is cleared by the failing check
    x = torch.randn((64, 128), device=ctx.device)
    g = torch.ones(128, device=ctx.device)
    y = ctx.layernorm(x, g, torch.zeros(128, device=ctx.device), 1e-6)
    ctx.check()
    ref = torch.nn.functional.layer_norm(x, (128,), g, None, 1e-6)
    assert (y.float() - ref).abs().max() < 2e-2


def test_vit_forward_in_a_cuda_graph(ctx):
    """vit_forward only enqueues work on the given stream (kernels, memset, device copies), so after one
    warm-up call it can be captured in a CUDA graph; the replay reproduces the direct call bit for bit."""
    arch = synth.vit_tiny(layers=3, dim=128, heads=2, hidden=256, patch=4)
    gh, gw, B = 16, 20, 2
    full = dict(arch, attn_mode=synth.ATTN_SPARSE, block=8, radius=1, filter_layer=1, keep_ratio=0.5)
    w = synth.vit_weights(11, arch, gh, gw, pos_base=4)
    dw = ctx.make_vit_weights(w)
    dev = ctx.device
    img = torch.from_numpy(synth.tissue_batch(12, B, gh * 4, gw * 4)).to(dev)
    out, kept = ctx.vit_forward(full, dw, img, gh, gw)
    ctx.check()
    ref, ref_kept = out.clone(), kept.clone()      # (the context's cached workspace is reused by the captured call)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(graph, stream=s):
            out2, kept2 = ctx.vit_forward(full, dw, img, gh, gw, out=out, stream=s)
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    ctx.check()
    assert torch.equal(out, ref)
    assert torch.equal(kept2, ref_kept)
