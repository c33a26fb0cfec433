"""Pins of the oracle's whole forward: an independent fp64 restatement with library ops on tiny
models, plus structural identities (dense == sparse when the radius covers the grid, keep 1.0 ==
no filter, zero LayerScale == LayerNorm of the embeddings)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
import synth


def _torch_forward(arch, cfg, w, image, gh, gw, forced_keep=None):
    """fp64 library-op restatement (conv patch embedding, F.layer_norm, F.linear, F.gelu, SDPA)."""
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    D, G, P, H = arch["dim"], arch["n_global"], arch["patch"], arch["heads"]
    img = t(image)
    B = img.shape[0]
    x = F.conv2d(img, t(w["w_pe"]).reshape(D, 3, P, P), t(w["b_pe"]), stride=P)
    x = x.flatten(2).transpose(1, 2)
    x = torch.cat([t(w["cls"])[None].expand(B, -1, -1), x], 1) + t(w["pos"])[None]
    pos = torch.arange(gh * gw)[None].expand(B, -1)
    kept = None
    # filter stages written out here, independently of the oracle's helpers: (layer, keep ratio) pairs
    stages = list(cfg.get("filters") or
                  ([(cfg["filter_layer"], cfg["keep_ratio"])] if cfg.get("filter_layer", 0) > 0 else []))
    kept_positions, taken = [], 0
    for li, lw in enumerate(w["layers"], start=1):
        N = x.shape[1]
        h = F.layer_norm(x, (D,), t(lw["ln1_g"]), t(lw["ln1_b"]), arch["ln_eps"])
        qkv = F.linear(h, t(lw["w_qkv"]), t(lw["b_qkv"])).reshape(B, N, 3, H, D // H)
        q, k, v = (qkv[:, :, i].transpose(1, 2) for i in range(3))
        mask = torch.ones(B, 1, N, N, dtype=torch.bool)
        if cfg["attn_mode"] == synth.ATTN_SPARSE:
            by, bx = (pos // gw) // cfg["block"], (pos % gw) // cfg["block"]
            near = ((by[:, :, None] - by[:, None]).abs() <= cfg["radius"]) & \
                   ((bx[:, :, None] - bx[:, None]).abs() <= cfg["radius"])
            mask[:, 0, G:, G:] = near
        s = (q @ k.transpose(-1, -2)) / (D // H) ** 0.5
        s = s.masked_fill(~mask, float("-inf"))
        p = s.softmax(-1)
        a = (p @ v).transpose(1, 2).reshape(B, N, D)
        a = F.linear(a, t(lw["w_o"]), t(lw["b_o"]))
        x = x + (t(lw["ls1"]) * a if "ls1" in lw else a)
        h = F.layer_norm(x, (D,), t(lw["ln2_g"]), t(lw["ln2_b"]), arch["ln_eps"])
        u = F.linear(h, t(lw["w_fc1"]), t(lw["b_fc1"]))
        if arch["mlp_kind"] == synth.MLP_SWIGLU:
            u = F.silu(u) * F.linear(h, t(lw["w_fc3"]), t(lw["b_fc3"]))
        else:
            u = F.gelu(u)
        m = F.linear(u, t(lw["w_fc2"]), t(lw["b_fc2"]))
        x = x + (t(lw["ls2"]) * m if "ls2" in lw else m)
        for layer, ratio in stages:
            if li != layer:
                continue
            npatch = N - G
            kk = int(np.ceil(ratio * npatch - 1e-9))
            if forced_keep is not None:
                # original positions of this stage's survivors -> indices among the tokens present
                want = torch.from_numpy(np.asarray(forced_keep)[:, taken:taken + kk]).long()
                kept = torch.stack([torch.searchsorted(pos[b].contiguous(), want[b]) for b in range(B)])
                assert bool((torch.gather(pos, 1, kept) == want).all())
            else:
                score = p[:, :, 0, G:].to(torch.float32).mean(1)
                order = torch.argsort(-score.double(), dim=-1, stable=True)[:, :kk]
                kept = torch.sort(order, dim=-1).values
            idx = torch.cat([torch.arange(G)[None].expand(B, -1), kept + G], 1)
            x = torch.gather(x, 1, idx[:, :, None].expand(-1, -1, D))
            pos = torch.gather(pos, 1, kept)
            kept_positions.append(pos.clone())
            taken += kk
    out = F.layer_norm(x, (D,), t(w["lnf_g"]), t(w["lnf_b"]), arch["ln_eps"])
    return out.numpy(), None if not kept_positions else torch.cat(kept_positions, 1).numpy()


def _setup(arch, gh, gw, seed=0, batch=2):
    w = synth.vit_weights(seed, arch, gh, gw, pos_base=4)
    img = synth.tissue_batch(seed + 1, batch, gh * arch["patch"], gw * arch["patch"])
    return w, img


@pytest.mark.parametrize("gh,gw,kind,ls,G", [(8, 8, synth.MLP_GELU, 1, 1), (9, 7, synth.MLP_SWIGLU, 0, 1),
                                             (6, 10, synth.MLP_GELU, 1, 2)])
def test_forward_matches_library_restatement(gh, gw, kind, ls, G):
    arch = synth.vit_tiny(layers=3, dim=64, heads=2, hidden=96, patch=4, mlp_kind=kind,
                          layerscale=ls, n_global=G)
    w, img = _setup(arch, gh, gw)
    cfg = dict(arch, attn_mode=synth.ATTN_SPARSE, block=2, radius=1, filter_layer=1, keep_ratio=0.6)
    got = oracle.vit_forward(cfg, w, img, gh, gw)
    want, wkept = _torch_forward(arch, cfg, w, img, gh, gw, forced_keep=got["kept_idx"])
    assert np.abs(got["out"] - want).max() < 2e-5
    # free-running ranking agrees as well unless two scores are closer than fp32 resolution
    want2, wkept2 = _torch_forward(arch, cfg, w, img, gh, gw)
    if np.array_equal(wkept2, got["kept_idx"]):
        assert np.abs(got["out"] - want2).max() < 2e-5
    assert got["out"].shape == (2, G + oracle.keep_count(gh * gw, 0.6), 64)


@pytest.mark.parametrize("gh,gw,kind,stages", [
    (8, 8, synth.MLP_GELU, [(1, 0.6), (3, 0.5)]),
    (9, 7, synth.MLP_SWIGLU, [(2, 0.75), (3, 0.4)]),
    (10, 6, synth.MLP_GELU, [(1, 0.8), (2, 0.7), (4, 0.5)]),
])
def test_forward_with_several_filter_stages(gh, gw, kind, stages):
    """Sec. 3.3 applied more than once: every stage ranks the tokens still present by that block's CLS
    attention, survivors keep their original grid positions for the neighbourhood rule of Sec. 3.2."""
    arch = synth.vit_tiny(layers=4, dim=64, heads=2, hidden=96, patch=4, mlp_kind=kind, layerscale=1)
    w, img = _setup(arch, gh, gw, seed=11)
    cfg = dict(arch, attn_mode=synth.ATTN_SPARSE, block=2, radius=1, filters=stages)
    got = oracle.vit_forward(cfg, w, img, gh, gw)
    counts, cur = [], gh * gw
    for _, ratio in stages:
        cur = int(np.ceil(ratio * cur - 1e-9))
        counts.append(cur)
    assert got["kept_all"].shape == (2, sum(counts)) and got["out"].shape == (2, 1 + counts[-1], 64)
    # every stage's set is ascending, and a subset of the stage before
    off, prev = 0, None
    for c in counts:
        seg = got["kept_all"][:, off:off + c]
        assert (np.diff(seg, axis=1) > 0).all()
        if prev is not None:
            assert all(set(seg[b]) <= set(prev[b]) for b in range(2))
        prev, off = seg, off + c
    assert np.array_equal(got["kept_idx"], prev)
    # teacher-forced with the oracle's own sets, the library restatement gives the same tokens
    want, _ = _torch_forward(arch, cfg, w, img, gh, gw, forced_keep=got["kept_all"])
    assert np.abs(got["out"] - want).max() < 2e-5
    # and the oracle, forced with its own sets, reproduces itself exactly
    again = oracle.vit_forward(cfg, w, img, gh, gw, forced_keep=got["kept_all"])
    assert np.array_equal(again["out"], got["out"])
    # free-running restatement: same sets unless two scores are closer than fp32 resolution
    want2, wkept2 = _torch_forward(arch, cfg, w, img, gh, gw)
    if np.array_equal(wkept2, got["kept_all"]):
        assert np.abs(got["out"] - want2).max() < 2e-5
    # one stage through the list form == the single-stage fields
    one = oracle.vit_forward(dict(cfg, filters=stages[:1]), w, img, gh, gw)
    legacy = dict(cfg, filter_layer=stages[0][0], keep_ratio=stages[0][1])
    legacy.pop("filters")
    assert np.array_equal(one["out"], oracle.vit_forward(legacy, w, img, gh, gw)["out"])


def test_forward_dense_mode_and_structural_identities():
    arch = synth.vit_tiny(layers=2, dim=64, heads=2, hidden=128, patch=4)
    gh, gw = 8, 6
    w, img = _setup(arch, gh, gw, seed=3)
    dense = dict(arch, attn_mode=synth.ATTN_DENSE, block=2, radius=0)
    cover = dict(arch, attn_mode=synth.ATTN_SPARSE, block=2, radius=3)
    local = dict(arch, attn_mode=synth.ATTN_SPARSE, block=2, radius=0)
    od = oracle.vit_forward(dense, w, img, gh, gw)["out"]
    want, _ = _torch_forward(arch, dense, w, img, gh, gw)
    assert np.abs(od - want).max() < 2e-5
    oc = oracle.vit_forward(cover, w, img, gh, gw)["out"]
    assert np.abs(od - oc).max() < 1e-6                       # radius covers the grid == dense
    ol = oracle.vit_forward(local, w, img, gh, gw)["out"]
    assert np.abs(od - ol).max() > 1e-4                       # and a real restriction differs
    # keep ratio 1.0 == no filter
    k1 = oracle.vit_forward(dict(local, filter_layer=1, keep_ratio=1.0), w, img, gh, gw)
    assert np.array_equal(k1["out"], ol)
    assert k1["kept_idx"].tolist() == [list(range(gh * gw))] * 2
    # zero LayerScale: every block is switched off, output = final LN of the embeddings
    wz = dict(w, layers=[dict(l, ls1=np.zeros(64, np.float32), ls2=np.zeros(64, np.float32))
                         for l in w["layers"]])
    oz = oracle.vit_forward(local, wz, img, gh, gw, tap_layer=0)
    assert np.abs(oz["out"] - oracle.layernorm(oz["tap"], w["lnf_g"], w["lnf_b"], 1e-6)).max() < 1e-6


def test_building_blocks_against_library():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 48)).astype(np.float32)
    w = rng.standard_normal((20, 48)).astype(np.float32)
    b = rng.standard_normal(20).astype(np.float32)
    assert np.abs(oracle.linear(x, w, b) - (x.astype(np.float64) @ w.T.astype(np.float64) + b)).max() < 1e-5
    g = rng.standard_normal(48).astype(np.float32)
    be = rng.standard_normal(48).astype(np.float32)
    ref = F.layer_norm(torch.from_numpy(x).double(), (48,), torch.from_numpy(g).double(),
                       torch.from_numpy(be).double(), 1e-6).numpy()
    assert np.abs(oracle.layernorm(x, g, be, 1e-6) - ref).max() < 1e-5
    for v in (-3.0, -0.5, 0.0, 0.7, 4.0):
        assert abs(oracle.gelu(v) - float(F.gelu(torch.tensor(v, dtype=torch.float64)))) < 1e-6
        assert abs(oracle.silu(v) - float(F.silu(torch.tensor(v, dtype=torch.float64)))) < 1e-6
    # the array forms of the two activations (what the timed CPU baseline loops over)
    a = rng.standard_normal(1000).astype(np.float32) * 3
    g2 = rng.standard_normal(1000).astype(np.float32)
    ta, tg = torch.from_numpy(a).double(), torch.from_numpy(g2).double()
    assert np.abs(oracle.gelu_n(a) - F.gelu(ta).numpy()).max() < 1e-6
    assert np.abs(oracle.silu_mul_n(a, g2) - (F.silu(ta) * tg).numpy()).max() < 2e-6
