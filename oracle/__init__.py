"""ctypes binding of the CPU oracle (test infrastructure).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library never does.  Arrays are numpy, host memory, fp32 unless
stated.  Each function cites the passage its C routine follows.
"""
import ctypes as C
import numpy as np

from .build import build as _build

_lib = None

MLP_GELU, MLP_SWIGLU = 0, 1
ATTN_DENSE, ATTN_SPARSE = 0, 1


class _AttnDesc(C.Structure):
    _fields_ = [("batch", C.c_int32), ("grid_h", C.c_int32), ("grid_w", C.c_int32),
                ("block", C.c_int32), ("radius", C.c_int32), ("n_global", C.c_int32),
                ("heads", C.c_int32), ("head_dim", C.c_int32), ("softmax_scale", C.c_float),
                ("n_patch", C.c_int32), ("patch_pos", C.c_void_p)]


class _VitConfig(C.Structure):
    _fields_ = [("layers", C.c_int32), ("dim", C.c_int32), ("heads", C.c_int32),
                ("mlp_hidden", C.c_int32), ("mlp_kind", C.c_int32), ("patch", C.c_int32),
                ("n_global", C.c_int32), ("has_layerscale", C.c_int32), ("ln_eps", C.c_float),
                ("attn_mode", C.c_int32), ("block", C.c_int32), ("radius", C.c_int32),
                ("filter_layer", C.c_int32), ("keep_ratio", C.c_double),
                ("n_filters", C.c_int32), ("filter_layers", C.c_int32 * 4), ("keep_ratios", C.c_double * 4)]


_LAYER_FIELDS = ["ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o", "ls1", "ln2_g", "ln2_b",
                 "w_fc1", "b_fc1", "w_fc3", "b_fc3", "w_fc2", "b_fc2", "ls2"]


class _LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _LAYER_FIELDS]


class _VitWeights(C.Structure):
    _fields_ = [("w_pe", C.c_void_p), ("b_pe", C.c_void_p), ("cls", C.c_void_p),
                ("pos", C.c_void_p), ("lnf_g", C.c_void_p), ("lnf_b", C.c_void_p),
                ("layer", C.c_void_p)]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build())
        _lib.spvo_gelu.restype = C.c_float
        _lib.spvo_gelu.argtypes = [C.c_float]
        _lib.spvo_silu.restype = C.c_float
        _lib.spvo_silu.argtypes = [C.c_float]
        _lib.spvo_keep_count.argtypes = [C.c_int32, C.c_double]
        _lib.spvo_gelu_n.restype = None
        _lib.spvo_silu_mul_n.restype = None
        _lib.spvo_layernorm.restype = None
        _lib.spvo_linear.restype = None
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def num_threads():
    return int(lib().spvo_num_threads())


def _desc(batch, grid_h, grid_w, block, radius, n_global, heads, head_dim, n_patch,
          patch_pos, scale):
    d = _AttnDesc(batch, grid_h, grid_w, block, radius, n_global, heads, head_dim,
                  float(scale), n_patch, _ptr(patch_pos))
    return d


def mask(grid_h, grid_w, block, radius, n_global=1, patch_pos=None):
    """Sec. 3.2: boolean [N, N] matrix of allowed (query, key) pairs for one image."""
    pp = None if patch_pos is None else np.ascontiguousarray(patch_pos, dtype=np.int32)
    n_patch = grid_h * grid_w if pp is None else pp.shape[-1]
    d = _desc(1, grid_h, grid_w, block, radius, n_global, 1, 1, n_patch, pp, 0.0)
    n = n_global + n_patch
    f = lib().spvo_allowed
    out = np.zeros((n, n), dtype=bool)
    for i in range(n):
        for j in range(n):
            out[i, j] = bool(f(C.byref(d), 0, i, j))
    return out


def attention(q, k, v, grid_h, grid_w, block, radius, n_global=1, patch_pos=None,
              scale=0.0, rows=None, want_scores=False):
    """Sec. 3.2 masked attention; q, k, v fp32 [B, N, h, e].  Returns (o, cls_scores|None).

    With `rows` (int32 list of query token indices) only those rows of o are filled."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    B, N, H, E = q.shape
    pp = None if patch_pos is None else np.ascontiguousarray(patch_pos, dtype=np.int32)
    n_patch = N - n_global
    if pp is not None:
        assert pp.shape == (B, n_patch)
    else:
        assert n_patch == grid_h * grid_w
    d = _desc(B, grid_h, grid_w, block, radius, n_global, H, E, n_patch, pp, scale)
    o = np.zeros_like(q)
    sc = np.zeros((B, H, n_patch), dtype=np.float32) if want_scores else None
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int32)
    rc = lib().spvo_attention(C.byref(d), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(sc),
                              _ptr(r), C.c_int32(0 if r is None else r.size))
    if rc != 0:
        raise ValueError(f"spvo_attention failed ({rc})")
    return o, sc


def dense_attention(q, k, v, scale=0.0):
    """Textbook dense softmax attention; q, k, v fp32 [B, N, h, e]."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    B, N, H, E = q.shape
    o = np.zeros_like(q)
    lib().spvo_dense_attention(B, N, H, E, C.c_float(scale), _ptr(q), _ptr(k), _ptr(v), _ptr(o))
    return o


def keep_count(n_patch, keep_ratio):
    """Sec. 3.3: k = ceil(keep_ratio * n_patch)."""
    k = int(lib().spvo_keep_count(int(n_patch), float(keep_ratio)))
    if k < 0:
        raise ValueError("keep_ratio must be in (0, 1] and n_patch >= 1")
    return k


def token_filter(scores, tokens=None, n_global=1, keep_ratio=0.5):
    """Sec. 3.3 filter.  scores fp32 [B, h, n_patch]; tokens uint16 [B, G+n_patch, dim] or None.

    Returns (tokens_out | None, kept_idx int32 [B, k], mean fp32 [B, n_patch])."""
    scores = _f32(scores)
    B, H, NP = scores.shape
    k = keep_count(NP, keep_ratio)
    kept = np.zeros((B, k), dtype=np.int32)
    mean = np.zeros((B, NP), dtype=np.float32)
    tin = tout = None
    dim = 0
    if tokens is not None:
        tin = np.ascontiguousarray(tokens, dtype=np.uint16)
        assert tin.shape[:2] == (B, n_global + NP)
        dim = tin.shape[2]
        tout = np.zeros((B, n_global + k, dim), dtype=np.uint16)
    rc = lib().spvo_filter(B, H, NP, n_global, dim, C.c_double(keep_ratio), _ptr(scores),
                           _ptr(tin), _ptr(tout), _ptr(kept), _ptr(mean))
    if rc != 0:
        raise ValueError(f"spvo_filter failed ({rc})")
    return tout, kept, mean


def layernorm(x, g, b, eps):
    x, g, b = _f32(x), _f32(g), _f32(b)
    y = np.empty_like(x)
    rows = x.size // x.shape[-1]
    lib().spvo_layernorm(_ptr(x), C.c_int64(rows), C.c_int32(x.shape[-1]), _ptr(g), _ptr(b),
                         C.c_float(eps), _ptr(y))
    return y


def linear(x, w, bias=None):
    x, w = _f32(x), _f32(w)
    bias = None if bias is None else _f32(bias)
    rows = x.size // x.shape[-1]
    y = np.empty(x.shape[:-1] + (w.shape[0],), dtype=np.float32)
    lib().spvo_linear(_ptr(x), C.c_int64(rows), C.c_int32(x.shape[-1]), C.c_int32(w.shape[0]),
                      _ptr(w), _ptr(bias), _ptr(y))
    return y


def gelu(x):
    return float(lib().spvo_gelu(float(x)))


def silu(x):
    return float(lib().spvo_silu(float(x)))


def gelu_n(a):
    """Exact (erf) GELU over an array."""
    a = _f32(a)
    y = np.empty_like(a)
    lib().spvo_gelu_n(_ptr(a), C.c_int64(a.size), _ptr(y))
    return y


def silu_mul_n(a, b):
    """silu(a) * b over arrays (the SwiGLU gate)."""
    a, b = _f32(a), _f32(b)
    y = np.empty_like(a)
    lib().spvo_silu_mul_n(_ptr(a), _ptr(b), C.c_int64(a.size), _ptr(y))
    return y


def filter_stages(cfg):
    """[(layer, keep_ratio), ...] of a config dict: `filters` (a list of such pairs, layers strictly
    increasing) or the single stage `filter_layer` / `keep_ratio`."""
    if cfg.get("filters"):
        return [(int(l), float(k)) for l, k in cfg["filters"]]
    if cfg.get("filter_layer", 0) > 0:
        return [(int(cfg["filter_layer"]), float(cfg["keep_ratio"]))]
    return []


def stage_keep_counts(cfg, npatch):
    """Tokens kept by each stage, in order."""
    out, cur = [], npatch
    for _, keep in filter_stages(cfg):
        cur = keep_count(cur, keep)
        out.append(cur)
    return out


def vit_forward(cfg, weights, image, grid_h, grid_w, forced_keep=None, tap_layer=None):
    """Whole forward.  cfg: dict with the spvo_vit_config fields (`filters`: optional list of
    (layer, keep_ratio) stages); weights: dict of fp32 numpy arrays (`w_pe, b_pe, cls, pos, lnf_g, lnf_b`
    and `layers`: list of dicts with the per-layer names); image fp32 [B, 3, H*patch, W*patch].
    forced_keep: [B, k_1 + ... + k_S] original positions kept by each stage, stage after stage.

    Returns dict(out=[B, G+k, dim], kept_idx=[B, k] of the last stage | None,
    kept_all=[B, k_1+...+k_S] | None, tap=... | None)."""
    image = _f32(image)
    B = image.shape[0]
    stages = filter_stages(cfg)
    multi = bool(cfg.get("filters"))
    fl = (C.c_int32 * 4)(*([l for l, _ in stages] + [0] * (4 - len(stages)))) if multi else (C.c_int32 * 4)()
    kr = (C.c_double * 4)(*([k for _, k in stages] + [0.0] * (4 - len(stages)))) if multi else (C.c_double * 4)()
    c = _VitConfig(cfg["layers"], cfg["dim"], cfg["heads"], cfg["mlp_hidden"], cfg["mlp_kind"],
                   cfg["patch"], cfg["n_global"], cfg.get("has_layerscale", 0),
                   cfg.get("ln_eps", 1e-6), cfg["attn_mode"], cfg.get("block", 8),
                   cfg.get("radius", 1), 0 if multi else cfg.get("filter_layer", 0),
                   1.0 if multi else cfg.get("keep_ratio", 1.0), len(stages) if multi else 0, fl, kr)
    keepalive = []

    def fp(a):
        if a is None:
            return None
        a = _f32(a)
        keepalive.append(a)
        return _ptr(a)

    L = (_LayerWeights * cfg["layers"])()
    for i, lw in enumerate(weights["layers"]):
        for n in _LAYER_FIELDS:
            setattr(L[i], n, fp(lw.get(n)))
    w = _VitWeights(fp(weights["w_pe"]), fp(weights["b_pe"]), fp(weights["cls"]),
                    fp(weights["pos"]), fp(weights["lnf_g"]), fp(weights["lnf_b"]),
                    C.cast(L, C.c_void_p))
    G, D = cfg["n_global"], cfg["dim"]
    npatch = grid_h * grid_w
    counts = stage_keep_counts(cfg, npatch)
    k = counts[-1] if counts else npatch
    k_total = sum(counts)
    out = np.zeros((B, G + k, D), dtype=np.float32)
    kept = np.zeros((B, k_total), dtype=np.int32) if counts else None
    fk = None
    if forced_keep is not None:
        fk = np.ascontiguousarray(forced_keep, dtype=np.int32)
        assert fk.shape == (B, k_total)
    tap = None
    tl = -1
    if tap_layer is not None:
        tl = int(tap_layer)
        ntap = npatch
        for (layer, _), cnt in zip(stages, counts):
            if tl >= layer:
                ntap = cnt
        tap = np.zeros((B, G + ntap, D), dtype=np.float32)
    rc = lib().spvo_vit_forward(C.byref(c), C.byref(w), _ptr(image), B, grid_h, grid_w, _ptr(out),
                                _ptr(kept), _ptr(fk), C.c_int32(tl), _ptr(tap))
    if rc != 0:
        raise ValueError(f"spvo_vit_forward failed ({rc})")
    return {"out": out, "kept_idx": None if kept is None else kept[:, k_total - k:], "kept_all": kept, "tap": tap}
