"""Thin Python binding of libspatvit (argument marshalling only).

Every step of the path runs inside the CUDA library; PyTorch is used for device memory and
streams.  The library must have been built (`python -m paper_2601_12150_b200.build` or
`__graft_entry__.build()`); importing the compute entry points without it raises.
There is no CPU fallback.
"""
import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspatvit.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_ALIGNMENT, ERR_STATIC_LIMIT = range(8)
FILTER_STATIC_BYTES = 2 << 20
TOKENS_ROW_MAJOR, TOKENS_BLOCK_MAJOR = 0, 1
MLP_GELU, MLP_SWIGLU = 0, 1
ATTN_DENSE, ATTN_SPARSE = 0, 1
EPI_BIAS, EPI_BIAS_GELU, EPI_BIAS_SILU, EPI_BIAS_MUL, EPI_BIAS_SCALE_RESID, EPI_BIAS_ADDROW = range(6)

EXPORTS = ["spv_create", "spv_destroy", "spv_status_string", "spv_check", "spv_last_wait_site", "spv_launch_count",
           "spv_attn_workspace_size", "spatial_block_attention",
           "spv_filter_keep_count", "spv_filter_workspace_size", "cls_score_topk_filter",
           "cls_score_topk_filter_static",
           "spv_vit_workspace_size", "vit_forward", "spv_gemm_bf16", "spv_layernorm",
           "spv_profile_enable", "spv_profile_read", "spv_microbench", "spv_selftest_wait"]


class SpvError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


class AttnDesc(C.Structure):
    _fields_ = [("batch", C.c_int32), ("grid_h", C.c_int32), ("grid_w", C.c_int32),
                ("block", C.c_int32), ("radius", C.c_int32), ("n_global", C.c_int32),
                ("heads", C.c_int32), ("head_dim", C.c_int32), ("softmax_scale", C.c_float),
                ("n_patch", C.c_int32), ("patch_pos", C.c_void_p), ("token_order", C.c_int32),
                ("stride_b", C.c_int64), ("stride_tok", C.c_int64), ("stride_head", C.c_int64)]


class FilterDesc(C.Structure):
    _fields_ = [("batch", C.c_int32), ("heads", C.c_int32), ("n_patch", C.c_int32),
                ("n_global", C.c_int32), ("dim", C.c_int32), ("keep_ratio", C.c_double),
                ("in_stride_b", C.c_int64), ("out_stride_b", C.c_int64)]


class VitConfig(C.Structure):
    _fields_ = [("layers", C.c_int32), ("dim", C.c_int32), ("heads", C.c_int32),
                ("mlp_hidden", C.c_int32), ("mlp_kind", C.c_int32), ("patch", C.c_int32),
                ("n_global", C.c_int32), ("has_layerscale", C.c_int32), ("ln_eps", C.c_float),
                ("attn_mode", C.c_int32), ("block", C.c_int32), ("radius", C.c_int32),
                ("filter_layer", C.c_int32), ("keep_ratio", C.c_double),
                ("n_filters", C.c_int32), ("filter_layers", C.c_int32 * 4), ("keep_ratios", C.c_double * 4),
                ("unfused_filter", C.c_int32)]


LAYER_FIELDS = ["ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o", "ls1", "ln2_g", "ln2_b",
                "w_fc1", "b_fc1", "w_fc3", "b_fc3", "w_fc2", "b_fc2", "ls2"]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in LAYER_FIELDS]


class VitWeights(C.Structure):
    _fields_ = [("w_pe", C.c_void_p), ("b_pe", C.c_void_p), ("cls", C.c_void_p),
                ("pos", C.c_void_p), ("lnf_g", C.c_void_p), ("lnf_b", C.c_void_p),
                ("layer", C.c_void_p)]


KERNEL_CLASSES = ["gemm", "attn_patch", "attn_global", "attn_plan", "layernorm", "filter_select",
                  "filter_gather", "misc"]


class KernelStat(C.Structure):
    _fields_ = [("launches", C.c_int64), ("ms", C.c_double), ("work", C.c_double)]


class GemmDesc(C.Structure):
    _fields_ = [("m", C.c_int32), ("n", C.c_int32), ("k", C.c_int32),
                ("lda", C.c_int64), ("ldw", C.c_int64), ("ldo", C.c_int64),
                ("epilogue", C.c_int32), ("bias", C.c_void_p), ("aux", C.c_void_p),
                ("ldaux", C.c_int64), ("scale", C.c_void_p), ("addrow", C.c_void_p),
                ("ldadd", C.c_int64), ("rows_per_image", C.c_int32)]


MICROBENCH_KINDS = {"ex2": 0, "softmax_body": 1, "mma_ss": 2, "mma_ts": 3, "l2_tma": 4}


class MicrobenchDesc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("ctas_per_sm", C.c_int32), ("threads", C.c_int32), ("iters", C.c_int32),
                ("m", C.c_int32), ("n", C.c_int32), ("box_rows", C.c_int32), ("stages", C.c_int32),
                ("poly_per_8", C.c_int32), ("accumulators", C.c_int32),
                ("issue_mode", C.c_int32), ("issuers", C.c_int32)]


class MicrobenchResult(C.Structure):
    _fields_ = [("ms", C.c_double), ("cycles", C.c_double), ("units", C.c_double), ("sm_count", C.c_int32)]


_lib = None


def lib():
    """The loaded C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build the CUDA library first "
                               "(python -m paper_2601_12150_b200.build); there is no fallback path")
        L = C.CDLL(LIB_PATH)
        L.spv_status_string.restype = C.c_char_p
        L.spv_status_string.argtypes = [C.c_int32]
        L.spv_launch_count.restype = C.c_int64
        L.spv_launch_count.argtypes = [C.c_void_p]
        L.spv_last_wait_site.restype = C.c_uint32
        L.spv_last_wait_site.argtypes = [C.c_void_p]
        L.spv_create.argtypes = [C.POINTER(C.c_void_p), C.c_int32]
        L.spv_destroy.argtypes = [C.c_void_p]
        L.spv_check.argtypes = [C.c_void_p, C.c_void_p]
        L.spv_filter_keep_count.argtypes = [C.c_int32, C.c_double, C.POINTER(C.c_int32)]
        L.spv_filter_workspace_size.argtypes = [C.POINTER(FilterDesc), C.POINTER(C.c_size_t)]
        L.cls_score_topk_filter.argtypes = [C.c_void_p, C.POINTER(FilterDesc)] + [C.c_void_p] * 8 + \
            [C.c_size_t, C.c_void_p]
        L.cls_score_topk_filter_static.argtypes = [C.POINTER(FilterDesc)] + [C.c_void_p] * 8
        L.spv_attn_workspace_size.argtypes = [C.POINTER(AttnDesc), C.POINTER(C.c_size_t)]
        L.spatial_block_attention.argtypes = [C.c_void_p, C.POINTER(AttnDesc)] + [C.c_void_p] * 6 + \
            [C.c_size_t, C.c_void_p]
        L.spv_vit_workspace_size.argtypes = [C.POINTER(VitConfig), C.c_int32, C.c_int32, C.c_int32,
                                             C.POINTER(C.c_size_t)]
        L.vit_forward.argtypes = [C.c_void_p, C.POINTER(VitConfig), C.POINTER(VitWeights), C.c_void_p,
                                  C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.c_size_t, C.c_void_p]
        L.spv_gemm_bf16.argtypes = [C.c_void_p, C.POINTER(GemmDesc), C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.c_void_p]
        L.spv_layernorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p,
                                    C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]
        L.spv_profile_enable.argtypes = [C.c_void_p, C.c_int32]
        L.spv_profile_read.argtypes = [C.c_void_p, C.POINTER(KernelStat)]
        L.spv_selftest_wait.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
        L.spv_microbench.argtypes = [C.c_void_p, C.POINTER(MicrobenchDesc), C.c_void_p, C.c_size_t, C.c_void_p,
                                     C.POINTER(MicrobenchResult)]
        _lib = L
    return _lib


def status_string(status):
    return lib().spv_status_string(int(status)).decode()


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _raise(status, what):
    if status != OK:
        raise SpvError(status, what)


def filter_keep_count(n_patch, keep_ratio):
    k = C.c_int32(0)
    _raise(lib().spv_filter_keep_count(int(n_patch), float(keep_ratio), C.byref(k)), "spv_filter_keep_count")
    return k.value


def cls_score_topk_filter_static(scores, tokens_in, tokens_out, kept_idx, n_global=1, keep_ratio=0.5,
                                 mean_scores=None, pos_in=None, pos_out=None, stream=None):
    """The token filter through the entry point that allocates nothing: no context, no workspace
    (its scratch is a 2 MiB array built into the library), and this wrapper creates no tensor
    either -- every output is the caller's.  For callers that run under a fixed device-memory
    plan or inside a loop where an allocation would stall the device.  Works on the current CUDA
    device; calls that may overlap on the GPU must be ordered by the caller (shared scratch).
    scores fp32 [B, h, n_patch]; tokens_in / tokens_out bf16 [B, G+n_patch, dim] / [B, G+k, dim] or
    both None; kept_idx int32 [B, k]."""
    import torch
    B, H, NP = scores.shape
    dim = 0 if tokens_in is None else tokens_in.shape[-1]
    d = FilterDesc(B, H, NP, n_global, dim, float(keep_ratio), 0, 0)
    # the library writes k rows / indices per image into the caller's buffers: a buffer of another size, type or
    # device would be written out of bounds, so check them here (the count fails below if the ratio is invalid)
    kc = C.c_int32(0)
    if lib().spv_filter_keep_count(NP, float(keep_ratio), C.byref(kc)) == OK:
        k = kc.value
        dev = scores.device
        assert scores.dtype == torch.float32 and scores.is_contiguous()
        assert kept_idx.dtype == torch.int32 and kept_idx.is_contiguous() and tuple(kept_idx.shape) == (B, k)
        assert kept_idx.device == dev
        if tokens_in is not None:
            assert tokens_out is not None and tokens_in.dtype == tokens_out.dtype == torch.bfloat16
            assert tokens_in.is_contiguous() and tokens_out.is_contiguous()
            assert tuple(tokens_in.shape) == (B, n_global + NP, dim) and tuple(tokens_out.shape) == (B, n_global + k, dim)
            assert tokens_in.device == dev and tokens_out.device == dev
        if mean_scores is not None:
            assert mean_scores.dtype == torch.float32 and mean_scores.is_contiguous() and tuple(mean_scores.shape) == (B, NP)
        if pos_in is not None:
            assert pos_out is not None and pos_in.dtype == pos_out.dtype == torch.int32
            assert tuple(pos_in.shape) == (B, NP) and tuple(pos_out.shape) == (B, k)
            assert pos_in.is_contiguous() and pos_out.is_contiguous()
    with torch.cuda.device(scores.device):
        st = lib().cls_score_topk_filter_static(C.byref(d), _ptr(scores), _ptr(tokens_in), _ptr(tokens_out),
                                                _ptr(kept_idx), _ptr(mean_scores), _ptr(pos_in), _ptr(pos_out),
                                                _stream(stream))
    _raise(st, "cls_score_topk_filter_static")
    return tokens_out, kept_idx


class Context:
    """Owns an spv_ctx for one CUDA device and the workspaces it hands to the library."""

    def __init__(self, device=0):
        import torch
        self._torch = torch
        self.device = torch.device("cuda", device)
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _raise(lib().spv_create(C.byref(h), device), "spv_create")
        self.handle = h
        self._ws = None

    def close(self):
        if self.handle:
            lib().spv_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace(self, nbytes):
        """A cached device workspace of at least `nbytes` (grown on demand, 256-byte aligned)."""
        torch = self._torch
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = None
            self._ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=self.device)
        return self._ws

    def check(self, stream=None):
        st = lib().spv_check(self.handle, _stream(stream))
        if st == ERR_TIMEOUT:
            raise SpvError(st, "spv_check (wait site 0x%x)" % lib().spv_last_wait_site(self.handle))
        _raise(st, "spv_check")

    def launch_count(self):
        return int(lib().spv_launch_count(self.handle))

    def profile(self, enable=True):
        """Start (and clear) or stop the per-kernel-class event timing."""
        _raise(lib().spv_profile_enable(self.handle, 1 if enable else 0), "spv_profile_enable")

    def profile_read(self):
        """{class: dict(launches, ms, work)} accumulated since the last read; waits for the events."""
        arr = (KernelStat * len(KERNEL_CLASSES))()
        _raise(lib().spv_profile_read(self.handle, arr), "spv_profile_read")
        return {n: dict(launches=int(a.launches), ms=float(a.ms), work=float(a.work))
                for n, a in zip(KERNEL_CLASSES, arr)}

    def microbench(self, kind, ctas_per_sm=1, threads=128, iters=1000, m=128, n=64, box_rows=64, stages=4,
                   poly_per_8=0, accumulators=1, issue_mode=0, issuers=1, stream=None):
        """One hardware rate probe (spv_microbench); returns dict(ms, cycles, units, sm_count)."""
        d = MicrobenchDesc(MICROBENCH_KINDS[kind], ctas_per_sm, threads, iters, m, n, box_rows, stages, poly_per_8,
                           accumulators, issue_mode, issuers)
        nbytes = (32 << 20) + (64 << 10) if kind == "l2_tma" else (64 << 10)
        buf = self.workspace(nbytes)
        r = MicrobenchResult()
        _raise(lib().spv_microbench(self.handle, C.byref(d), _ptr(buf), buf.numel(), _stream(stream), C.byref(r)),
               "spv_microbench")
        return dict(ms=r.ms, cycles=r.cycles, units=r.units, sm_count=r.sm_count)

    # -- Sec. 3.3 ---------------------------------------------------------------------------
    def cls_score_topk_filter(self, scores, tokens_in=None, n_global=1, keep_ratio=0.5,
                              tokens_out=None, kept_idx=None, mean_scores=None, pos_in=None,
                              pos_out=None, workspace=None, stream=None):
        """scores fp32 [B, h, n_patch]; tokens_in bf16 [B, G+n_patch, dim] or None.
        Returns (tokens_out | None, kept_idx int32 [B, k])."""
        torch = self._torch
        B, H, NP = scores.shape
        k = filter_keep_count(NP, keep_ratio)
        dim = 0 if tokens_in is None else tokens_in.shape[-1]
        d = FilterDesc(B, H, NP, n_global, dim, float(keep_ratio), 0, 0)
        if kept_idx is None:
            kept_idx = torch.empty((B, k), dtype=torch.int32, device=scores.device)
        if tokens_in is not None and tokens_out is None:
            tokens_out = torch.empty((B, n_global + k, dim), dtype=tokens_in.dtype, device=scores.device)
        if workspace is None:
            need = C.c_size_t(0)
            _raise(lib().spv_filter_workspace_size(C.byref(d), C.byref(need)), "spv_filter_workspace_size")
            workspace = self.workspace(need.value)
        st = lib().cls_score_topk_filter(self.handle, C.byref(d), _ptr(scores), _ptr(tokens_in),
                                         _ptr(tokens_out), _ptr(kept_idx), _ptr(mean_scores), _ptr(pos_in),
                                         _ptr(pos_out), _ptr(workspace), workspace.numel(), _stream(stream))
        _raise(st, "cls_score_topk_filter")
        return tokens_out, kept_idx

    # -- Sec. 3.2 ---------------------------------------------------------------------------
    def attn_desc(self, q, grid_h, grid_w, block, radius, n_global=1, patch_pos=None, scale=0.0,
                  token_order=TOKENS_ROW_MAJOR):
        B, N, H, E = q.shape
        sb, st, sh, se = q.stride()
        assert se == 1
        return AttnDesc(B, grid_h, grid_w, block, radius, n_global, H, E, float(scale), N - n_global,
                        None if patch_pos is None else patch_pos.data_ptr(), token_order, sb, st, sh)

    def spatial_block_attention(self, q, k, v, grid_h, grid_w, block, radius, n_global=1, patch_pos=None,
                                scale=0.0, token_order=TOKENS_ROW_MAJOR, out=None, want_scores=False,
                                workspace=None, stream=None):
        """q, k, v bf16 [B, N, h, 64] views with identical strides.  Returns (o, cls_scores | None)."""
        torch = self._torch
        assert q.stride() == k.stride() == v.stride()
        d = self.attn_desc(q, grid_h, grid_w, block, radius, n_global, patch_pos, scale, token_order)
        if out is None:
            out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=q.device)
        assert out.stride() == q.stride()
        sc = None
        if want_scores:
            sc = torch.empty((q.shape[0], q.shape[2], q.shape[1] - n_global), dtype=torch.float32,
                             device=q.device)
        if workspace is None:
            need = C.c_size_t(0)
            _raise(lib().spv_attn_workspace_size(C.byref(d), C.byref(need)), "spv_attn_workspace_size")
            workspace = self.workspace(need.value)
        st = lib().spatial_block_attention(self.handle, C.byref(d), _ptr(q), _ptr(k), _ptr(v), _ptr(out),
                                           _ptr(sc), _ptr(workspace), workspace.numel(), _stream(stream))
        _raise(st, "spatial_block_attention")
        return out, sc

    # -- building blocks ----------------------------------------------------------------------
    def gemm_bf16(self, a, w, out, epilogue=EPI_BIAS, bias=None, aux=None, scale=None, addrow=None,
                  rows_per_image=0, stream=None):
        """out = epilogue(a [M, K] @ w [N, K]^T); see spv_gemm_desc in include/spatvit.h."""
        M, K = a.shape
        N = w.shape[0]
        d = GemmDesc(M, N, K, a.stride(0), w.stride(0), out.stride(0), epilogue,
                     None if bias is None else bias.data_ptr(),
                     None if aux is None else aux.data_ptr(), 0 if aux is None else aux.stride(0),
                     None if scale is None else scale.data_ptr(),
                     None if addrow is None else addrow.data_ptr(),
                     0 if addrow is None else addrow.stride(0), rows_per_image)
        _raise(lib().spv_gemm_bf16(self.handle, C.byref(d), _ptr(a), _ptr(w), _ptr(out), _stream(stream)),
               "spv_gemm_bf16")
        return out

    def layernorm(self, x, gamma, beta, eps=1e-6, out=None, out_row=None, stream=None):
        torch = self._torch
        rows, dim = x.shape
        if out is None:
            out = torch.empty((rows, dim), dtype=torch.bfloat16, device=x.device)
        _raise(lib().spv_layernorm(self.handle, _ptr(x), rows, dim, _ptr(gamma), _ptr(beta), float(eps),
                                   _ptr(out), _ptr(out_row), _stream(stream)), "spv_layernorm")
        return out

    # -- Sec. 3 / 4.1 ---------------------------------------------------------------------------
    def make_vit_weights(self, weights):
        """Upload a dict of numpy fp32 weights (synth.vit_weights layout): matrices as bf16, vectors
        as fp32.  Returns an object holding the device tensors and the C structs."""
        return VitWeightsOnDevice(self, weights)

    def vit_forward(self, cfg, dev_weights, image, grid_h, grid_w, forced_keep=None, want_kept=True,
                    out=None, workspace=None, stream=None):
        """cfg: dict with the spv_vit_config fields; `filters`: optional list of (layer, keep_ratio) stages
        in place of filter_layer / keep_ratio.  image fp32 device [B, 3, H*p, W*p].  forced_keep: int32
        device [B, k_1 + ... + k_S] (the layout of the returned kept array).
        Returns (out_tokens bf16 [B, G+k, dim], kept int32 [B, k_1 + ... + k_S] | None)."""
        torch = self._torch
        stages = vit_filter_stages(cfg)
        multi = bool(cfg.get("filters"))
        fl = (C.c_int32 * 4)(*([l for l, _ in stages] + [0] * (4 - len(stages)))) if multi else (C.c_int32 * 4)()
        kr = (C.c_double * 4)(*([r for _, r in stages] + [0.0] * (4 - len(stages)))) if multi else (C.c_double * 4)()
        c = VitConfig(cfg["layers"], cfg["dim"], cfg["heads"], cfg["mlp_hidden"], cfg["mlp_kind"],
                      cfg["patch"], cfg["n_global"], cfg.get("has_layerscale", 0), cfg.get("ln_eps", 1e-6),
                      cfg["attn_mode"], cfg.get("block", 8), cfg.get("radius", 1),
                      0 if multi else cfg.get("filter_layer", 0), 1.0 if multi else cfg.get("keep_ratio", 1.0),
                      len(stages) if multi else 0, fl, kr, int(cfg.get("unfused_filter", 0)))
        B = image.shape[0]
        npatch = grid_h * grid_w
        counts, cur = [], npatch
        for _, ratio in stages:
            cur = filter_keep_count(cur, ratio)
            counts.append(cur)
        k = counts[-1] if counts else npatch
        if out is None:
            out = torch.empty((B, cfg["n_global"] + k, cfg["dim"]), dtype=torch.bfloat16, device=image.device)
        kept = torch.empty((B, sum(counts)), dtype=torch.int32, device=image.device) if (counts and want_kept) else None
        if forced_keep is not None:
            assert forced_keep.dtype == torch.int32 and forced_keep.is_contiguous()
            assert tuple(forced_keep.shape) == (B, sum(counts)), "forced_keep: one row of k_1 + ... + k_S per image"
        if workspace is None:
            need = C.c_size_t(0)
            _raise(lib().spv_vit_workspace_size(C.byref(c), B, grid_h, grid_w, C.byref(need)),
                   "spv_vit_workspace_size")
            workspace = self.workspace(need.value)
        st = lib().vit_forward(self.handle, C.byref(c), C.byref(dev_weights.struct), _ptr(image), B, grid_h,
                               grid_w, _ptr(out), _ptr(kept), _ptr(forced_keep), _ptr(workspace),
                               workspace.numel(), _stream(stream))
        _raise(st, "vit_forward")
        return out, kept

    def selftest_wait(self, limit_ns=200000, stream=None):
        """Launch the library's one-CTA kernel that waits on a barrier nobody arrives on; the wait gives up
        after limit_ns and the next check() reports the expired wait."""
        _raise(lib().spv_selftest_wait(self.handle, int(limit_ns), _stream(stream)), "spv_selftest_wait")


def vit_filter_stages(cfg):
    """[(layer, keep_ratio), ...] of a config dict."""
    if cfg.get("filters"):
        return [(int(l), float(r)) for l, r in cfg["filters"]]
    if cfg.get("filter_layer", 0) > 0:
        return [(int(cfg["filter_layer"]), float(cfg["keep_ratio"]))]
    return []


class VitWeightsOnDevice:
    MATRICES = {"w_pe", "w_qkv", "w_o", "w_fc1", "w_fc2", "w_fc3"}

    def __init__(self, ctx, weights):
        import numpy as np
        import torch
        self.tensors = []

        def up(name, a):
            if a is None:
                return None
            t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(ctx.device)
            if name in self.MATRICES:
                t = t.to(torch.bfloat16)
            t = t.contiguous()
            self.tensors.append(t)
            return t.data_ptr()

        n = len(weights["layers"])
        self.layers = (LayerWeights * n)()
        for i, lw in enumerate(weights["layers"]):
            for f in LAYER_FIELDS:
                setattr(self.layers[i], f, up(f, lw.get(f)))
        self.struct = VitWeights(up("w_pe", weights["w_pe"]), up("b_pe", weights["b_pe"]),
                                 up("cls", weights["cls"]), up("pos", weights["pos"]),
                                 up("lnf_g", weights["lnf_g"]), up("lnf_b", weights["lnf_b"]),
                                 C.cast(self.layers, C.c_void_p))
