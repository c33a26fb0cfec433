"""Seeded synthetic inputs shaped like the paper's workloads.

These stand in for the pathology images and the pretrained backbone weights the
paper uses (neither is available): they reproduce shapes, token counts, value
ranges and the background fraction only.  This module holds NO arithmetic of the
method itself; it only draws data, rounds it to bf16 once, and hands the same
values to both the CUDA library and the CPU oracle.
"""
import numpy as np

# --------------------------------------------------------------------------- #
# bf16 <-> fp32 data conversion (round to nearest even), numpy only
# --------------------------------------------------------------------------- #


def f32_to_bf16_bits(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b):
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def round_bf16(a):
    """fp32 array whose values are exactly representable in bf16."""
    return bf16_bits_to_f32(f32_to_bf16_bits(a))


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _trunc_normal(rng, shape, std=0.02):
    z = rng.standard_normal(shape, dtype=np.float32)
    bad = np.abs(z) > 2.0
    while bad.any():
        z[bad] = rng.standard_normal(int(bad.sum()), dtype=np.float32)
        bad = np.abs(z) > 2.0
    return z * np.float32(std)


def _smooth_field(rng, h, w, cell):
    """Low-frequency random field in [0,1]-ish: coarse noise, bicubic upsampled."""
    import torch
    import torch.nn.functional as F
    gh, gw = max(2, h // cell + 2), max(2, w // cell + 2)
    coarse = torch.from_numpy(rng.standard_normal((1, 1, gh, gw), dtype=np.float32))
    up = F.interpolate(coarse, size=(h, w), mode="bicubic", align_corners=False)
    return up[0, 0].numpy()


# --------------------------------------------------------------------------- #
# single attention op (28x28 grid + CLS, 16 heads x 64)
# --------------------------------------------------------------------------- #


def attention_qkv(seed, batch, n_tok, heads, head_dim=64, std=1.0):
    """Q, K, V ~ N(0, std^2), three consecutive draws, rounded to bf16.

    Returns three fp32 arrays [batch, n_tok, heads, head_dim] holding bf16-exact values."""
    rng = _rng(seed)
    shape = (batch, n_tok, heads, head_dim)
    return tuple(round_bf16(rng.standard_normal(shape, dtype=np.float32) * np.float32(std))
                 for _ in range(3))


# --------------------------------------------------------------------------- #
# token-filter op (CLS->patch score tensor + token rows)
# --------------------------------------------------------------------------- #


def background_mask(rng, grid_h, grid_w, fraction, cell=8):
    """Spatially coherent boolean mask covering exactly round(fraction*H*W) positions."""
    f = _smooth_field(rng, grid_h, grid_w, cell).reshape(-1)
    n_bg = int(round(fraction * f.size))
    order = np.argsort(f, kind="stable")
    m = np.zeros(f.size, dtype=bool)
    m[order[:n_bg]] = True
    return m.reshape(grid_h, grid_w)


def filter_scores(seed, batch, heads, grid_h, grid_w, bg_fraction=0.35, tie_quantum=None):
    """CLS->patch softmax scores, fp32 [batch, heads, H*W].

    Logits are 2*N(0,1); a spatially coherent 35 % of the positions (shared by all heads of an
    image) is pushed down by 8 to mimic background; each head row is a softmax over the
    patches.  With `tie_quantum` the scores are snapped to multiples of it (tie stress)."""
    rng = _rng(seed)
    n = grid_h * grid_w
    logits = 2.0 * rng.standard_normal((batch, heads, n), dtype=np.float32)
    for b in range(batch):
        bg = background_mask(rng, grid_h, grid_w, bg_fraction).reshape(-1)
        logits[b][:, bg] -= 8.0
    z = logits.astype(np.float64)
    z -= z.max(axis=-1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=-1, keepdims=True)
    p = p.astype(np.float32)
    if tie_quantum is not None:
        p = (np.round(p / np.float32(tie_quantum)) * np.float32(tie_quantum)).astype(np.float32)
    return p


def token_rows(seed, batch, n_tok, dim):
    """bf16 token rows as uint16 bit patterns [batch, n_tok, dim], values ~ N(0,1)."""
    rng = _rng(seed)
    return f32_to_bf16_bits(rng.standard_normal((batch, n_tok, dim), dtype=np.float32))


# --------------------------------------------------------------------------- #
# ViT architectures, weights and tissue-like images
# --------------------------------------------------------------------------- #

MLP_GELU, MLP_SWIGLU = 0, 1
ATTN_DENSE, ATTN_SPARSE = 0, 1


def vit_l16():
    return dict(layers=24, dim=1024, heads=16, mlp_hidden=4096, mlp_kind=MLP_GELU, patch=16,
                n_global=1, has_layerscale=1, ln_eps=1e-6)


def vit_g14():
    return dict(layers=40, dim=1536, heads=24, mlp_hidden=4096, mlp_kind=MLP_SWIGLU, patch=14,
                n_global=1, has_layerscale=0, ln_eps=1e-6)


def vit_tiny(layers=2, dim=128, heads=2, hidden=256, patch=4, mlp_kind=MLP_GELU, layerscale=1,
             n_global=1):
    return dict(layers=layers, dim=dim, heads=heads, mlp_hidden=hidden, mlp_kind=mlp_kind,
                patch=patch, n_global=n_global, has_layerscale=layerscale, ln_eps=1e-6)


def interpolate_pos_embed(base, n_global, base_h, base_w, grid_h, grid_w):
    """Resize a learned position table [G + bh*bw, d] to [G + H*W, d] (bicubic on the grid).

    One-off host preprocessing of an input; both sides receive the result."""
    import torch
    import torch.nn.functional as F
    d = base.shape[1]
    g = base[:n_global]
    p = torch.from_numpy(base[n_global:].reshape(1, base_h, base_w, d)).permute(0, 3, 1, 2)
    p = F.interpolate(p, size=(grid_h, grid_w), mode="bicubic", align_corners=False)
    p = p.permute(0, 2, 3, 1).reshape(grid_h * grid_w, d).numpy()
    return np.concatenate([g, p], axis=0).astype(np.float32)


def vit_weights(seed, arch, grid_h, grid_w, pos_base=14, layerscale_init=0.1):
    """Random-init weights (trunc-normal std 0.02 matrices), every value bf16-exact fp32.

    Matrices follow the [out_features, in_features] convention.  Vectors: biases N(0, 0.02),
    LayerNorm gamma 1 + N(0, 0.05), beta N(0, 0.02), LayerScale `layerscale_init`*(1 + N(0,0.1))
    (not 1e-5: that would switch every block off and make parity vacuous)."""
    rng = _rng(seed)
    D, HID, P, G = arch["dim"], arch["mlp_hidden"], arch["patch"], arch["n_global"]

    def mat(o, i):
        return round_bf16(_trunc_normal(rng, (o, i)))

    def vec(n, mean=0.0, std=0.02):
        return round_bf16(np.float32(mean) + np.float32(std) * rng.standard_normal(n, dtype=np.float32))

    w = {"w_pe": mat(D, 3 * P * P), "b_pe": vec(D), "cls": round_bf16(_trunc_normal(rng, (G, D)))}
    base = _trunc_normal(rng, (G + pos_base * pos_base, D))
    w["pos"] = round_bf16(interpolate_pos_embed(base, G, pos_base, pos_base, grid_h, grid_w))
    w["lnf_g"], w["lnf_b"] = vec(D, 1.0, 0.05), vec(D)
    layers = []
    for _ in range(arch["layers"]):
        lw = {"ln1_g": vec(D, 1.0, 0.05), "ln1_b": vec(D),
              "w_qkv": mat(3 * D, D), "b_qkv": vec(3 * D),
              "w_o": mat(D, D), "b_o": vec(D),
              "ln2_g": vec(D, 1.0, 0.05), "ln2_b": vec(D),
              "w_fc1": mat(HID, D), "b_fc1": vec(HID),
              "w_fc2": mat(D, HID), "b_fc2": vec(D)}
        if arch["mlp_kind"] == MLP_SWIGLU:
            lw["w_fc3"], lw["b_fc3"] = mat(HID, D), vec(HID)
        if arch["has_layerscale"]:
            lw["ls1"] = vec(D, layerscale_init, 0.1 * layerscale_init)
            lw["ls2"] = vec(D, layerscale_init, 0.1 * layerscale_init)
        layers.append(lw)
    w["layers"] = layers
    return w


_MEAN = np.array([0.485, 0.456, 0.406], dtype=np.float32)
_STD = np.array([0.229, 0.224, 0.225], dtype=np.float32)


def tissue_image(rng, size_h, size_w, background=0.4):
    """One H&E-like image, fp32 [3, size_h, size_w], channel-normalised.

    Tissue = thresholded low-frequency noise covering (1 - background) of the area, pink with
    darker purple nuclei-like blobs; background close to white; Gaussian pixel noise."""
    low = _smooth_field(rng, size_h, size_w, cell=max(32, min(size_h, size_w) // 8))
    thr = np.quantile(low[::4, ::4], background)
    tissue = low > thr
    mid = _smooth_field(rng, size_h, size_w, cell=6)
    nuclei = np.clip((mid - 0.6) * 1.5, 0.0, 1.0)
    pink = np.array([0.91, 0.62, 0.78], dtype=np.float32)
    purple = np.array([0.42, 0.25, 0.60], dtype=np.float32)
    white = np.array([0.96, 0.95, 0.96], dtype=np.float32)
    img = np.empty((3, size_h, size_w), dtype=np.float32)
    for ch in range(3):
        t = pink[ch] + (purple[ch] - pink[ch]) * nuclei
        img[ch] = np.where(tissue, t, white[ch])
    img += 0.02 * rng.standard_normal(img.shape, dtype=np.float32)
    np.clip(img, 0.0, 1.0, out=img)
    img = (img - _MEAN[:, None, None]) / _STD[:, None, None]
    return img.astype(np.float32)


def tissue_batch(seed, batch, size_h, size_w, background=0.4, background_range=None):
    """fp32 [batch, 3, size_h, size_w]; background fraction fixed or uniform in a range."""
    rng = _rng(seed)
    out = np.empty((batch, 3, size_h, size_w), dtype=np.float32)
    for b in range(batch):
        bg = background if background_range is None else float(rng.uniform(*background_range))
        out[b] = tissue_image(rng, size_h, size_w, bg)
    return out
