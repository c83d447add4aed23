"""ctypes binding of libssconv.so: the same entry points as include/ssconv.h.

Only argument marshalling happens here; torch supplies device memory and the current
stream.  There is no CPU path: if the library is missing or a call fails, an exception
is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Tuple

import torch

FLAG_BIAS = 1
FLAG_RELU = 2
FLAG_GELU = 4
MASK_LOGITS_F32 = 0
MASK_MAGNITUDE_BF16 = 1
MASK_MAGNITUDE_E4M3 = 2
OK = 0
ERR_TIMEOUT = 8

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libssconv.so")
EXPORTS = ("ssconv_version", "ssconv_launch_count", "ssconv_status_string", "ssconv_out_shape", "ssconv_sizes",
           "ssconv_plan", "ssconv_plan_for_sms", "ssconv_tune", "ssconv_window_extent", "ssconv_selftest_wait_timeout",
           "ssconv_select_mask", "ssconv_nm_patterns", "ssconv_select_mask_nm", "ssconv_apply_mask_nm",
           "ssconv_compress", "ssconv_decompress", "ssconv_maxpool", "ssconv_pad_channels", "ssconv_space_to_depth", "ssconv_unfold_w",
           "ssconv_fold_factor", "ssconv_fold_desc", "ssconv_fold_weights", "ssconv_forward", "ssconv_forward_res",
           "ssconv_forward_dense_res", "ssconv_forward_dense", "ssconv_forward_dense_strided",
           "ssconv_mask_norms", "ssconv_absmax", "ssconv_stability_threshold", "ssconv_soft_mask", "ssconv_mask_grad", "ssconv_adamw", "ssconv_dgrad_prepare", "ssconv_dgrad_spread", "ssconv_wgrad", "ssconv_wgrad_ws_bytes", "ssconv_dgrad", "ssconv_dgrad_ws_bytes",
           "ssconv_forward_static_ws",
           "ssconv_sizes_grouped", "ssconv_compress_grouped", "ssconv_forward_grouped", "ssconv_forward_dense_grouped",
           "ssconv_depthwise", "ssconv_layernorm",
           "ssconv_quantize_e4m3", "ssconv_sizes_fp8", "ssconv_compress_fp8", "ssconv_decompress_fp8",
           "ssconv_forward_fp8", "ssconv_forward_dense_fp8")


class SsconvError(RuntimeError):
    def __init__(self, fn: str, status: int, text: str):
        super().__init__(f"{fn} failed: status {status} ({text})")
        self.status = status


class Desc(ctypes.Structure):
    """Mirror of ssconv_desc_t."""
    _fields_ = [(n, ctypes.c_int32) for n in (
        "N", "H", "W", "C_in", "C_out", "KH", "KW", "stride_h", "stride_w", "pad_h", "pad_w", "dil_h", "dil_w")] + [
        ("flags", ctypes.c_uint32)]


def make_desc(N, H, W, C_in, C_out, KH, KW, stride=1, pad=0, dil=1, bias=True, relu=False, gelu=False) -> Desc:
    def pair(v):
        return (v, v) if isinstance(v, int) else tuple(v)
    (sh, sw), (ph, pw), (dh, dw) = pair(stride), pair(pad), pair(dil)
    flags = (FLAG_BIAS if bias else 0) | (FLAG_RELU if relu else 0) | (FLAG_GELU if gelu else 0)
    return Desc(N, H, W, C_in, C_out, KH, KW, sh, sw, ph, pw, dh, dw, flags)


def desc_from_spec(spec) -> Desc:
    """Descriptor for a synth.LayerSpec."""
    return make_desc(spec.N, spec.H, spec.W, spec.C_in, spec.C_out, spec.KH, spec.KW, spec.stride, spec.pad,
                     spec.dil, bias=spec.has_bias, relu=spec.relu and not spec.gelu, gelu=spec.gelu)


_lib = None


def lib():
    """Load libssconv.so once; raise if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise FileNotFoundError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2411_00288_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        dp = ctypes.POINTER(Desc)
        L.ssconv_version.restype = i32
        L.ssconv_version.argtypes = []
        L.ssconv_launch_count.restype = ctypes.c_uint64
        L.ssconv_launch_count.argtypes = []
        L.ssconv_status_string.restype = ctypes.c_char_p
        L.ssconv_status_string.argtypes = [i32]
        L.ssconv_out_shape.restype = i32
        L.ssconv_out_shape.argtypes = [dp, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.ssconv_sizes.restype = i32
        L.ssconv_sizes.argtypes = [dp, ctypes.POINTER(i64)] + [ctypes.POINTER(sz)] * 4
        L.ssconv_select_mask.restype = i32
        L.ssconv_select_mask.argtypes = [i32, vp, i64, vp, vp]
        L.ssconv_compress.restype = i32
        L.ssconv_compress.argtypes = [dp, vp, vp, vp, vp, vp]
        L.ssconv_decompress.restype = i32
        L.ssconv_decompress.argtypes = [dp, vp, vp, vp, vp, vp]
        L.ssconv_forward.restype = i32
        L.ssconv_forward.argtypes = [dp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.ssconv_forward_dense.restype = i32
        L.ssconv_forward_dense.argtypes = [dp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.ssconv_forward_static_ws.restype = i32
        L.ssconv_forward_static_ws.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().ssconv_status_string(status).decode()


def _check(fn: str, status: int):
    if status != OK:
        raise SsconvError(fn, status, status_string(status))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _need_cuda(*tensors):
    for t in tensors:
        if t is not None and not (t.is_cuda and t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")


def ssconv_version() -> int:
    return int(lib().ssconv_version())


def ssconv_launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(lib().ssconv_launch_count())


def ssconv_out_shape(desc: Desc) -> Tuple[int, int]:
    h, w = ctypes.c_int32(), ctypes.c_int32()
    _check("ssconv_out_shape", lib().ssconv_out_shape(ctypes.byref(desc), ctypes.byref(h), ctypes.byref(w)))
    return int(h.value), int(w.value)


@dataclass(frozen=True)
class Sizes:
    G: int
    w_comp_bytes: int
    meta_bytes: int
    ws_bytes_sparse: int
    ws_bytes_dense: int


def ssconv_sizes(desc: Desc) -> Sizes:
    G = ctypes.c_int64()
    a, b, c, d = (ctypes.c_size_t() for _ in range(4))
    _check("ssconv_sizes", lib().ssconv_sizes(ctypes.byref(desc), ctypes.byref(G), ctypes.byref(a), ctypes.byref(b),
                                              ctypes.byref(c), ctypes.byref(d)))
    return Sizes(int(G.value), int(a.value), int(b.value), int(c.value), int(d.value))


def ssconv_select_mask(mode: int, scores: torch.Tensor, G: int, pattern: Optional[torch.Tensor] = None,
                       stream=None) -> torch.Tensor:
    """pattern uint8 [G] from fp32 scores [G,6] (mode LOGITS) or bf16 weights (mode MAGNITUDE)."""
    _need_cuda(scores, pattern)
    if pattern is None:
        pattern = torch.empty((G,), dtype=torch.uint8, device=scores.device)
    _check("ssconv_select_mask", lib().ssconv_select_mask(mode, _ptr(scores), G, _ptr(pattern), _stream(stream)))
    return pattern


def ssconv_nm_patterns(N: int, M: int) -> int:
    """n = C(M, N), the number of N:M patterns (0 if N, M are out of the supported range)."""
    f = lib().ssconv_nm_patterns
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_int32, ctypes.c_int32]
    return int(f(int(N), int(M)))


def ssconv_select_mask_nm(mode: int, scores: torch.Tensor, G: int, N: int, M: int, stream=None) -> torch.Tensor:
    """pattern uint8 [G] for N:M blocks from fp32 scores [G, n] (mode LOGITS) or bf16 weights [G, M] (MAGNITUDE)."""
    _need_cuda(scores)
    pattern = torch.empty((G,), dtype=torch.uint8, device=scores.device)
    f = lib().ssconv_select_mask_nm
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_int32, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                  ctypes.c_void_p]
    _check("ssconv_select_mask_nm", f(mode, _ptr(scores), G, N, M, _ptr(pattern), _stream(stream)))
    return pattern


def ssconv_apply_mask_nm(w: torch.Tensor, pattern: torch.Tensor, N: int, M: int, stream=None) -> torch.Tensor:
    """M .* W for an N:M mask: bf16 weights of w's shape with the dropped positions zeroed."""
    _need_cuda(w, pattern)
    out = torch.empty_like(w)
    f = lib().ssconv_apply_mask_nm
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                  ctypes.c_void_p]
    _check("ssconv_apply_mask_nm", f(_ptr(w), _ptr(pattern), pattern.numel(), N, M, _ptr(out), _stream(stream)))
    return out


def ssconv_compress(desc: Desc, w: torch.Tensor, pattern: torch.Tensor, stream=None):
    """(w_comp, meta) uint8 blobs from bf16 weights [C_out,KH,KW,C_in] and pattern [G]."""
    _need_cuda(w, pattern)
    sz = ssconv_sizes(desc)
    w_comp = torch.empty((sz.w_comp_bytes,), dtype=torch.uint8, device=w.device)
    meta = torch.empty((sz.meta_bytes,), dtype=torch.uint8, device=w.device)
    _check("ssconv_compress", lib().ssconv_compress(ctypes.byref(desc), _ptr(w), _ptr(pattern), _ptr(w_comp),
                                                    _ptr(meta), _stream(stream)))
    return w_comp, meta


def ssconv_decompress(desc: Desc, w_comp: torch.Tensor, meta: torch.Tensor, want_pattern: bool = True, stream=None):
    """(w_masked bf16 [C_out,KH,KW,C_in], pattern uint8 [G] or None) read back from the blobs."""
    _need_cuda(w_comp, meta)
    sz = ssconv_sizes(desc)
    w_out = torch.empty((desc.C_out, desc.KH, desc.KW, desc.C_in), dtype=torch.bfloat16, device=w_comp.device)
    pat = torch.empty((sz.G,), dtype=torch.uint8, device=w_comp.device) if want_pattern else None
    _check("ssconv_decompress", lib().ssconv_decompress(ctypes.byref(desc), _ptr(w_comp), _ptr(meta), _ptr(w_out),
                                                        _ptr(pat), _stream(stream)))
    return w_out, pat


_workspaces = {}


def ssconv_window_extent(n: int, k: int, stride: int = 1, pad: int = 0, dil: int = 1) -> int:
    """Placements of a k-tap window along an axis of n elements, as the library computes them."""
    f = lib().ssconv_window_extent
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_int32] * 5
    return int(f(int(n), int(k), int(stride), int(pad), int(dil)))


def ssconv_plan_for_sms(desc: Desc, sparse: bool, sm_count: int) -> dict:
    """ssconv_plan for a device with `sm_count` SMs; host arithmetic only, no GPU needed."""
    out = [ctypes.c_int32(0) for _ in range(5)]
    f = lib().ssconv_plan_for_sms
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.c_int32, ctypes.c_int32] + [ctypes.POINTER(ctypes.c_int32)] * 5
    _check("ssconv_plan_for_sms", f(ctypes.byref(desc), 1 if sparse else 0, int(sm_count), *[ctypes.byref(o) for o in out]))
    return dict(tile_positions=out[0].value, split=bool(out[1].value), ctas=out[2].value, ring_groups=out[3].value,
                pair=bool(out[4].value))


def ssconv_selftest_wait_timeout(limit_cycles: int, dev_status: torch.Tensor, stream=None) -> None:
    """Launch the one-block kernel whose bounded wait runs out; it stores ERR_TIMEOUT to dev_status."""
    _need_cuda(dev_status)
    f = lib().ssconv_selftest_wait_timeout
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
    _check("ssconv_selftest_wait_timeout", f(int(limit_cycles), _ptr(dev_status), _stream(stream)))


def ssconv_plan(desc: Desc, sparse: bool = True) -> dict:
    """Tile width, K split, thread blocks and ring depth the forward call would use on the current device."""
    out = [ctypes.c_int32(0) for _ in range(5)]
    f = lib().ssconv_plan
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.c_int32] + [ctypes.POINTER(ctypes.c_int32)] * 5
    _check("ssconv_plan", f(ctypes.byref(desc), 1 if sparse else 0, *[ctypes.byref(o) for o in out]))
    return dict(tile_positions=out[0].value, split=bool(out[1].value), ctas=out[2].value, ring_groups=out[3].value,
                pair=bool(out[4].value))


TUNE_TILE_POSITIONS, TUNE_PAIR, TUNE_WGRAD_RANGES, TUNE_WGRAD_PAIR, TUNE_RESIDENT_WEIGHTS, TUNE_PAIR_TILES = 1, 2, 3, 4, 5, 6


def ssconv_tune(option: int, value: int) -> None:
    """Process-wide planner override: TUNE_TILE_POSITIONS (0 = automatic, or a multiple of 16 in [48, 240]),
    TUNE_PAIR (-1 automatic, 0 never, 1 wherever thread-block pairs apply), TUNE_PAIR_TILES (-1 automatic, 0 one
    position tile per work item of the pair kernel, 1 two wherever they fit), the others as the header says."""
    f = lib().ssconv_tune
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_int32, ctypes.c_int32]
    _check("ssconv_tune", f(int(option), int(value)))


def default_workspace(device) -> torch.Tensor:
    """One scratch buffer per device, shared by calls that pass ws=None.  It needs no initialisation
    (the kernels write every part before reading it), so stream-ordered calls can share it; calls
    on different streams that may overlap must pass their own."""
    dev = torch.device(device)
    key = dev.index if dev.index is not None else torch.cuda.current_device()
    if key not in _workspaces:
        nbytes = ssconv_sizes(make_desc(1, 8, 8, 8, 8, 1, 1)).ws_bytes_sparse
        _workspaces[key] = torch.empty((nbytes,), dtype=torch.uint8, device=torch.device("cuda", key))
    return _workspaces[key]


def _alloc_y(desc: Desc, x: torch.Tensor) -> torch.Tensor:
    ho, wo = ssconv_out_shape(desc)
    return torch.empty((desc.N, ho, wo, desc.C_out), dtype=torch.bfloat16, device=x.device)


def ssconv_forward(desc: Desc, x: torch.Tensor, w_comp: torch.Tensor, meta: torch.Tensor,
                   bias: Optional[torch.Tensor] = None, y: Optional[torch.Tensor] = None,
                   ws: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                   stream=None, residual: Optional[torch.Tensor] = None) -> torch.Tensor:
    """2:4 masked convolution forward; returns y bf16 [N,H_out,W_out,C_out] (enqueued, not synchronised).
    With `residual` (bf16, the shape of y) the call is ssconv_forward_res: y = act(bias + conv + residual)."""
    _need_cuda(x, w_comp, meta, bias, y, ws, dev_status, residual)
    if y is None:
        y = _alloc_y(desc, x)
    if ws is None:
        ws = default_workspace(x.device)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    if residual is None:
        _check("ssconv_forward", lib().ssconv_forward(
            ctypes.byref(desc), _ptr(x), _ptr(w_comp), _ptr(meta), _ptr(bias), _ptr(y), _ptr(ws), ws_bytes,
            _ptr(dev_status), _stream(stream)))
    else:
        assert residual.shape == y.shape and residual.dtype == torch.bfloat16 and residual.is_contiguous()
        f = lib().ssconv_forward_res
        f.restype = ctypes.c_int32
        f.argtypes = [ctypes.POINTER(Desc)] + [ctypes.c_void_p] * 7 + [ctypes.c_size_t, ctypes.c_void_p,
                                                                     ctypes.c_void_p]
        _check("ssconv_forward_res", f(ctypes.byref(desc), _ptr(x), _ptr(w_comp), _ptr(meta), _ptr(bias),
                                       _ptr(residual), _ptr(y), _ptr(ws), ws_bytes, _ptr(dev_status),
                                       _stream(stream)))
    return y


def ssconv_forward_dense(desc: Desc, x: torch.Tensor, w: torch.Tensor, bias: Optional[torch.Tensor] = None,
                         y: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None,
                         dev_status: Optional[torch.Tensor] = None, stream=None,
                         residual: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Dense counterpart with bf16 weights [C_out,KH,KW,C_in]; `residual` as in ssconv_forward."""
    _need_cuda(x, w, bias, y, ws, dev_status, residual)
    if y is None:
        y = _alloc_y(desc, x)
    if ws is None:
        ws = default_workspace(x.device)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    if residual is None:
        _check("ssconv_forward_dense", lib().ssconv_forward_dense(
            ctypes.byref(desc), _ptr(x), _ptr(w), _ptr(bias), _ptr(y), _ptr(ws), ws_bytes, _ptr(dev_status),
            _stream(stream)))
    else:
        assert residual.shape == y.shape and residual.dtype == torch.bfloat16 and residual.is_contiguous()
        f = lib().ssconv_forward_dense_res
        f.restype = ctypes.c_int32
        f.argtypes = [ctypes.POINTER(Desc)] + [ctypes.c_void_p] * 6 + [ctypes.c_size_t, ctypes.c_void_p,
                                                                     ctypes.c_void_p]
        _check("ssconv_forward_dense_res", f(ctypes.byref(desc), _ptr(x), _ptr(w), _ptr(bias), _ptr(residual),
                                             _ptr(y), _ptr(ws), ws_bytes, _ptr(dev_status), _stream(stream)))
    return y


def ssconv_maxpool(x: torch.Tensor, k: int = 3, stride: int = 2, pad: int = 1, y: Optional[torch.Tensor] = None,
                   stream=None) -> torch.Tensor:
    """k x k max-pooling of NHWC bf16 activations; returns y [N,H_out,W_out,C] (enqueued, not synchronised)."""
    _need_cuda(x, y)
    n, h, w, c = x.shape
    if y is None:
        y = torch.empty((n, ssconv_window_extent(h, k, stride, pad), ssconv_window_extent(w, k, stride, pad), c),
                        dtype=torch.bfloat16, device=x.device)
    f = lib().ssconv_maxpool
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int32] * 7 + [ctypes.c_void_p]
    _check("ssconv_maxpool", f(_ptr(x), _ptr(y), n, h, w, c, k, stride, pad, _stream(stream)))
    return y


def ssconv_space_to_depth(x: torch.Tensor, block: int, pad: int, Hb: int, Wb: int, C_pad: int,
                          y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """y [N,Hb,Wb,C_pad] with y[n,r,q,(bh*block+bw)*C+c] = x[n, block*r-pad+bh, block*q-pad+bw, c] (zeros outside
    the image and in the padding channels) from x [N,H,W,C] bf16."""
    _need_cuda(x, y)
    n, h, w, c = x.shape
    if y is None:
        y = torch.empty((n, Hb, Wb, C_pad), dtype=torch.bfloat16, device=x.device)
    f = lib().ssconv_space_to_depth
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int32] * 9 + [ctypes.c_void_p]
    _check("ssconv_space_to_depth", f(_ptr(x), _ptr(y), n, h, w, c, block, pad, Hb, Wb, C_pad, _stream(stream)))
    return y


def ssconv_fold_factor(desc: Desc) -> int:
    """The number of neighbouring output pixels (1 or 2) the planner suggests folding into the output channels."""
    f = lib().ssconv_fold_factor
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc)]
    return int(f(ctypes.byref(desc)))


def ssconv_fold_desc(desc: Desc, f: int) -> Desc:
    """Descriptor of the layer with f output pixels of a row folded into f * C_out output channels."""
    out = Desc()
    fn = lib().ssconv_fold_desc
    fn.restype = ctypes.c_int32
    fn.argtypes = [ctypes.POINTER(Desc), ctypes.c_int32, ctypes.POINTER(Desc)]
    _check("ssconv_fold_desc", fn(ctypes.byref(desc), int(f), ctypes.byref(out)))
    return out


def ssconv_fold_weights(desc: Desc, f: int, w: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                        stream=None):
    """(w_folded, bias_folded) for ssconv_fold_desc(desc, f).  w: any tensor of C_out*KH*KW equal vectors (bf16 or
    e4m3 weights [C_out,KH,KW,C_in], patterns [G]); w_folded has the same dtype and f*C_out*KH*KW' vectors."""
    _need_cuda(w, bias)
    folded = ssconv_fold_desc(desc, f)
    w2 = b2 = None
    tap = 0
    if w is not None:
        vecs = desc.C_out * desc.KH * desc.KW
        assert w.is_contiguous() and w.numel() % vecs == 0
        per = w.numel() // vecs
        tap = per * w.element_size()
        w2 = torch.empty((folded.C_out, folded.KH, folded.KW, per), dtype=w.dtype, device=w.device)
        if w.dim() == 1:
            w2 = w2.view(-1)
    if bias is not None:
        assert bias.dtype == torch.float32
        b2 = torch.empty((folded.C_out,), dtype=torch.float32, device=bias.device)
    fn = lib().ssconv_fold_weights
    fn.restype = ctypes.c_int32
    fn.argtypes = [ctypes.POINTER(Desc), ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                   ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    _check("ssconv_fold_weights", fn(ctypes.byref(desc), int(f), _ptr(w), _ptr(w2), tap, _ptr(bias), _ptr(b2),
                                     _stream(stream)))
    return w2, b2


def ssconv_forward_dense_strided(desc: Desc, x: torch.Tensor, strides, w: torch.Tensor,
                                 bias: Optional[torch.Tensor] = None, y: Optional[torch.Tensor] = None,
                                 ws: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                                 stream=None) -> torch.Tensor:
    """ssconv_forward_dense on a strided (possibly overlapping) view of x: `strides` = element strides of
    (w, h, n); pixel (n, h, w) of the input the descriptor names starts n*s_n + h*s_h + w*s_w elements into x."""
    _need_cuda(x, w, bias, y, ws, dev_status)
    if y is None:
        y = _alloc_y(desc, x)
    if ws is None:
        ws = default_workspace(x.device)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    s_w, s_h, s_n = (int(v) for v in strides)
    f = lib().ssconv_forward_dense_strided
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                  ctypes.c_void_p, ctypes.c_void_p]
    _check("ssconv_forward_dense_strided", f(ctypes.byref(desc), _ptr(x), s_w, s_h, s_n, _ptr(w), _ptr(bias), _ptr(y),
                                             _ptr(ws), ws_bytes, _ptr(dev_status), _stream(stream)))
    return y


def ssconv_pad_channels(x: torch.Tensor, C_pad: int, y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Zero-pad the channels of x [..., C] bf16 to C_pad (a multiple of 8); returns y [..., C_pad]."""
    _need_cuda(x, y)
    *lead, c = x.shape
    pixels = 1
    for d in lead:
        pixels *= d
    if y is None:
        y = torch.empty((*lead, C_pad), dtype=torch.bfloat16, device=x.device)
    f = lib().ssconv_pad_channels
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]
    _check("ssconv_pad_channels", f(_ptr(x), _ptr(y), pixels, c, C_pad, _stream(stream)))
    return y


def ssconv_forward_static_ws(desc: Desc, x: torch.Tensor, w_comp: torch.Tensor, meta: torch.Tensor,
                             bias: Optional[torch.Tensor], y: torch.Tensor,
                             dev_status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """ssconv_forward with the library's built-in scratch: for callers that must not allocate device
    memory.  Nothing is allocated here either, so the caller passes the output tensor y.  Small
    layers only (at most 64 output tiles); calls that overlap on the GPU race on the shared scratch."""
    _need_cuda(x, w_comp, meta, bias, y, dev_status)
    _check("ssconv_forward_static_ws", lib().ssconv_forward_static_ws(
        ctypes.byref(desc), _ptr(x), _ptr(w_comp), _ptr(meta), _ptr(bias), _ptr(y), _ptr(dev_status),
        _stream(stream)))
    return y


# ----------------------------------------------------------------------------- grouped / depthwise / layer norm
def ssconv_sizes_grouped(desc: Desc, groups: int):
    G = ctypes.c_int64()
    a, b = ctypes.c_size_t(), ctypes.c_size_t()
    f = lib().ssconv_sizes_grouped
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.c_int32, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_size_t),
                  ctypes.POINTER(ctypes.c_size_t)]
    _check("ssconv_sizes_grouped", f(ctypes.byref(desc), groups, ctypes.byref(G), ctypes.byref(a), ctypes.byref(b)))
    return int(G.value), int(a.value), int(b.value)


def ssconv_compress_grouped(desc: Desc, groups: int, w: torch.Tensor, pattern: torch.Tensor, stream=None):
    """(w_comp, meta) of a grouped layer: the per-group blobs one after another."""
    _need_cuda(w, pattern)
    _, nv, nm = ssconv_sizes_grouped(desc, groups)
    w_comp = torch.empty((nv,), dtype=torch.uint8, device=w.device)
    meta = torch.empty((nm,), dtype=torch.uint8, device=w.device)
    f = lib().ssconv_compress_grouped
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.c_int32] + [ctypes.c_void_p] * 5
    _check("ssconv_compress_grouped", f(ctypes.byref(desc), groups, _ptr(w), _ptr(pattern), _ptr(w_comp), _ptr(meta),
                                        _stream(stream)))
    return w_comp, meta


def ssconv_forward_grouped(desc: Desc, groups: int, x: torch.Tensor, w_comp: torch.Tensor, meta: torch.Tensor,
                           bias: Optional[torch.Tensor] = None, y: Optional[torch.Tensor] = None,
                           dev_status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """2:4 masked grouped convolution (one launch per group on channel slices)."""
    _need_cuda(x, w_comp, meta, bias, y, dev_status)
    if y is None:
        y = _alloc_y(desc, x)
    ws = default_workspace(x.device)
    f = lib().ssconv_forward_grouped
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.c_int32] + [ctypes.c_void_p] * 6 + [ctypes.c_size_t, ctypes.c_void_p,
                                                                                  ctypes.c_void_p]
    _check("ssconv_forward_grouped", f(ctypes.byref(desc), groups, _ptr(x), _ptr(w_comp), _ptr(meta), _ptr(bias), _ptr(y),
                                       _ptr(ws), ws.numel(), _ptr(dev_status), _stream(stream)))
    return y


def ssconv_forward_dense_grouped(desc: Desc, groups: int, x: torch.Tensor, w: torch.Tensor,
                                 bias: Optional[torch.Tensor] = None, y: Optional[torch.Tensor] = None,
                                 dev_status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Dense grouped convolution; w bf16 [C_out, KH, KW, C_in/groups]."""
    _need_cuda(x, w, bias, y, dev_status)
    if y is None:
        y = _alloc_y(desc, x)
    ws = default_workspace(x.device)
    f = lib().ssconv_forward_dense_grouped
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.c_int32] + [ctypes.c_void_p] * 5 + [ctypes.c_size_t, ctypes.c_void_p,
                                                                                  ctypes.c_void_p]
    _check("ssconv_forward_dense_grouped", f(ctypes.byref(desc), groups, _ptr(x), _ptr(w), _ptr(bias), _ptr(y), _ptr(ws),
                                             ws.numel(), _ptr(dev_status), _stream(stream)))
    return y


def ssconv_depthwise(desc: Desc, x: torch.Tensor, w: torch.Tensor, bias: Optional[torch.Tensor] = None,
                     y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Dense depthwise convolution; w bf16 tap-major [KH, KW, C]."""
    _need_cuda(x, w, bias, y)
    if y is None:
        y = _alloc_y(desc, x)
    f = lib().ssconv_depthwise
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc)] + [ctypes.c_void_p] * 5
    _check("ssconv_depthwise", f(ctypes.byref(desc), _ptr(x), _ptr(w), _ptr(bias), _ptr(y), _stream(stream)))
    return y


def ssconv_layernorm(x: torch.Tensor, gamma: torch.Tensor, beta: torch.Tensor, eps: float = 1e-6,
                     y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Layer normalisation over the last axis of x (bf16), gamma / beta fp32 [C]."""
    _need_cuda(x, gamma, beta, y)
    c = x.shape[-1]
    if y is None:
        y = torch.empty_like(x)
    f = lib().ssconv_layernorm
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float, ctypes.c_void_p, ctypes.c_int64,
                  ctypes.c_int32, ctypes.c_void_p]
    _check("ssconv_layernorm", f(_ptr(x), _ptr(gamma), _ptr(beta), float(eps), _ptr(y), x.numel() // c, c, _stream(stream)))
    return y


# ----------------------------------------------------------------------------- 8-bit (e4m3) operands
def ssconv_quantize_e4m3(x: torch.Tensor, scale: float = 1.0, y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """uint8 e4m3 codes of x * scale (x bf16, an even number of elements), nearest even, saturating."""
    _need_cuda(x, y)
    assert x.dtype == torch.bfloat16
    if y is None:
        y = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
    f = lib().ssconv_quantize_e4m3
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_float, ctypes.c_void_p]
    _check("ssconv_quantize_e4m3", f(_ptr(x), _ptr(y), x.numel(), float(scale), _stream(stream)))
    return y


def ssconv_sizes_fp8(desc: Desc):
    """(G, w_comp_bytes, meta_bytes) of the e4m3 blobs."""
    G = ctypes.c_int64()
    a, b = ctypes.c_size_t(), ctypes.c_size_t()
    f = lib().ssconv_sizes_fp8
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_size_t),
                  ctypes.POINTER(ctypes.c_size_t)]
    _check("ssconv_sizes_fp8", f(ctypes.byref(desc), ctypes.byref(G), ctypes.byref(a), ctypes.byref(b)))
    return int(G.value), int(a.value), int(b.value)


def ssconv_compress_fp8(desc: Desc, w: torch.Tensor, pattern: torch.Tensor, stream=None):
    """(w_comp, meta) uint8 blobs from e4m3 weights [C_out,KH,KW,C_in] (uint8) and pattern [G]."""
    _need_cuda(w, pattern)
    _, nv, nm = ssconv_sizes_fp8(desc)
    w_comp = torch.empty((nv,), dtype=torch.uint8, device=w.device)
    meta = torch.empty((nm,), dtype=torch.uint8, device=w.device)
    f = lib().ssconv_compress_fp8
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc)] + [ctypes.c_void_p] * 5
    _check("ssconv_compress_fp8", f(ctypes.byref(desc), _ptr(w), _ptr(pattern), _ptr(w_comp), _ptr(meta), _stream(stream)))
    return w_comp, meta


def ssconv_decompress_fp8(desc: Desc, w_comp: torch.Tensor, meta: torch.Tensor, stream=None):
    """(w_masked uint8 e4m3 [C_out,KH,KW,C_in], pattern uint8 [G]) read back from the e4m3 blobs."""
    _need_cuda(w_comp, meta)
    G, _, _ = ssconv_sizes_fp8(desc)
    w_out = torch.empty((desc.C_out, desc.KH, desc.KW, desc.C_in), dtype=torch.uint8, device=w_comp.device)
    pat = torch.empty((G,), dtype=torch.uint8, device=w_comp.device)
    f = lib().ssconv_decompress_fp8
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc)] + [ctypes.c_void_p] * 5
    _check("ssconv_decompress_fp8", f(ctypes.byref(desc), _ptr(w_comp), _ptr(meta), _ptr(w_out), _ptr(pat), _stream(stream)))
    return w_out, pat


def ssconv_forward_fp8(desc: Desc, x: torch.Tensor, w_comp: torch.Tensor, meta: torch.Tensor,
                       bias: Optional[torch.Tensor] = None, out_scale: float = 1.0, y: Optional[torch.Tensor] = None,
                       dev_status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """2:4 masked convolution on e4m3 activations (uint8 NHWC) and compressed e4m3 weights; bf16 output."""
    _need_cuda(x, w_comp, meta, bias, y, dev_status)
    if y is None:
        y = _alloc_y(desc, x)
    f = lib().ssconv_forward_fp8
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc)] + [ctypes.c_void_p] * 4 + [ctypes.c_float] + [ctypes.c_void_p] * 3
    _check("ssconv_forward_fp8", f(ctypes.byref(desc), _ptr(x), _ptr(w_comp), _ptr(meta), _ptr(bias), float(out_scale),
                                   _ptr(y), _ptr(dev_status), _stream(stream)))
    return y


def ssconv_forward_dense_fp8(desc: Desc, x: torch.Tensor, w: torch.Tensor, bias: Optional[torch.Tensor] = None,
                             out_scale: float = 1.0, y: Optional[torch.Tensor] = None,
                             dev_status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Dense counterpart on e4m3 weights [C_out,KH,KW,C_in] (uint8)."""
    _need_cuda(x, w, bias, y, dev_status)
    if y is None:
        y = _alloc_y(desc, x)
    f = lib().ssconv_forward_dense_fp8
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc)] + [ctypes.c_void_p] * 3 + [ctypes.c_float] + [ctypes.c_void_p] * 3
    _check("ssconv_forward_dense_fp8", f(ctypes.byref(desc), _ptr(x), _ptr(w), _ptr(bias), float(out_scale), _ptr(y),
                                         _ptr(dev_status), _stream(stream)))
    return y


def ssconv_soft_mask(logits: torch.Tensor, noise: Optional[torch.Tensor], tau: float, w: Optional[torch.Tensor],
                     want_z: bool = True, want_w_eff: bool = True, stream=None,
                     z: Optional[torch.Tensor] = None, w_eff: Optional[torch.Tensor] = None):
    """(z fp32 [G,6] or None, w_eff bf16 shaped like w or None): relaxed choice (Eq. 3) and effective
    weights (Eq. 6 with the soft mask) of every group of four weights.  Output tensors may be passed in."""
    _need_cuda(logits, noise, w, z, w_eff)
    G = logits.shape[0]
    if z is None and want_z:
        z = torch.empty((G, 6), dtype=torch.float32, device=logits.device)
    if w_eff is None and want_w_eff:
        w_eff = torch.empty_like(w)
    f = lib().ssconv_soft_mask
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float, ctypes.c_void_p, ctypes.c_int64,
                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    _check("ssconv_soft_mask", f(_ptr(logits), _ptr(noise), float(tau), _ptr(w), G, _ptr(z), _ptr(w_eff),
                                 _stream(stream)))
    return z, w_eff


def ssconv_mask_grad(z: torch.Tensor, tau: float, w: torch.Tensor, g_w_eff: torch.Tensor,
                     g_logits: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """dL/dlogits fp32 [G,6] from dL/dw_eff (fp32, the shape of w)."""
    _need_cuda(z, w, g_w_eff, g_logits)
    G = z.shape[0]
    if g_logits is None:
        g_logits = torch.empty((G, 6), dtype=torch.float32, device=z.device)
    f = lib().ssconv_mask_grad
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p, ctypes.c_float, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                  ctypes.c_void_p, ctypes.c_void_p]
    _check("ssconv_mask_grad", f(_ptr(z), float(tau), _ptr(w), _ptr(g_w_eff), G, _ptr(g_logits), _stream(stream)))
    return g_logits


def ssconv_wgrad_ws_bytes(desc: Desc) -> int:
    n = ctypes.c_size_t()
    f = lib().ssconv_wgrad_ws_bytes
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.POINTER(ctypes.c_size_t)]
    _check("ssconv_wgrad_ws_bytes", f(ctypes.byref(desc), ctypes.byref(n)))
    return int(n.value)


def ssconv_wgrad(desc: Desc, x: torch.Tensor, dy: torch.Tensor, dw: Optional[torch.Tensor] = None,
                 ws: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                 stream=None) -> torch.Tensor:
    """Weight gradient fp32 [C_out,KH,KW,C_in] of the layer from its bf16 input x and output gradient dy."""
    _need_cuda(x, dy, dw, ws, dev_status)
    if dw is None:
        dw = torch.empty((desc.C_out, desc.KH, desc.KW, desc.C_in), dtype=torch.float32, device=x.device)
    if ws is None:
        need = ssconv_wgrad_ws_bytes(desc)
        ws = torch.empty((need,), dtype=torch.uint8, device=x.device) if need else None
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    f = lib().ssconv_wgrad
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                  ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p]
    _check("ssconv_wgrad", f(ctypes.byref(desc), _ptr(x), _ptr(dy), _ptr(dw), _ptr(ws), ws_bytes, _ptr(dev_status),
                             _stream(stream)))
    return dw


def ssconv_dgrad_ws_bytes(desc: Desc) -> int:
    n = ctypes.c_size_t()
    f = lib().ssconv_dgrad_ws_bytes
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.POINTER(ctypes.c_size_t)]
    _check("ssconv_dgrad_ws_bytes", f(ctypes.byref(desc), ctypes.byref(n)))
    return int(n.value)


def ssconv_dgrad(desc: Desc, dy: torch.Tensor, w: torch.Tensor, dx: Optional[torch.Tensor] = None,
                 ws: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                 stream=None) -> torch.Tensor:
    """Input gradient bf16 [N,H,W,C_in] of the layer from its output gradient dy and bf16 weights, any stride."""
    _need_cuda(dy, w, dx, ws, dev_status)
    if dx is None:
        dx = torch.empty((desc.N, desc.H, desc.W, desc.C_in), dtype=torch.bfloat16, device=dy.device)
    if ws is None:
        ws = torch.empty((max(ssconv_dgrad_ws_bytes(desc), 16),), dtype=torch.uint8, device=dy.device)
    f = lib().ssconv_dgrad
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                  ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p]
    _check("ssconv_dgrad", f(ctypes.byref(desc), _ptr(dy), _ptr(w), _ptr(dx), _ptr(ws), ws.numel() * ws.element_size(),
                             _ptr(dev_status), _stream(stream)))
    return dx


def ssconv_adamw(theta: torch.Tensor, g: torch.Tensor, m: torch.Tensor, v: torch.Tensor, step: int, lr: float = 1.0,
                 beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 1e-4,
                 stream=None) -> torch.Tensor:
    """One AdamW update of fp32 parameters in place (theta, m, v are modified); step counts from 1."""
    _need_cuda(theta, g, m, v)
    assert theta.dtype == g.dtype == m.dtype == v.dtype == torch.float32
    assert theta.numel() == g.numel() == m.numel() == v.numel()
    f = lib().ssconv_adamw
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int64, ctypes.c_int32] + [ctypes.c_float] * 5 + [ctypes.c_void_p]
    _check("ssconv_adamw", f(_ptr(theta), _ptr(g), _ptr(m), _ptr(v), theta.numel(), int(step), float(lr),
                             float(beta1), float(beta2), float(eps), float(weight_decay), _stream(stream)))
    return theta


def ssconv_unfold_w(x: torch.Tensor, KW: int, stride: int = 1, pad: int = 0, dil: int = 1, C_pad: Optional[int] = None,
                    y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Partial unfold along the width of x [..., W, C] bf16: y [..., W_out, C_pad] with
    y[..., wo, kw*C + c] = x[..., wo*stride - pad + kw*dil, c] (zeros outside and in padding channels)."""
    _need_cuda(x, y)
    *lead, w, c = x.shape
    rows = 1
    for d in lead:
        rows *= d
    if C_pad is None:
        C_pad = -(-KW * c // 64) * 64
    if y is None:
        y = torch.empty((*lead, ssconv_window_extent(w, KW, stride, pad, dil), C_pad), dtype=torch.bfloat16,
                        device=x.device)
    f = lib().ssconv_unfold_w
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64] + [ctypes.c_int32] * 7 + [ctypes.c_void_p]
    _check("ssconv_unfold_w", f(_ptr(x), _ptr(y), rows, w, c, KW, stride, pad, dil, C_pad, _stream(stream)))
    return y


LEMMA_PERTURBATION, LEMMA_ANY_MASK, LEMMA_MASKED_UPDATE = 34, 35, 36


def ssconv_mask_norms(w: torch.Tensor, pattern: torch.Tensor, out: Optional[torch.Tensor] = None,
                      stream=None) -> torch.Tensor:
    """fp32 [3] on the device: ||W||_inf, ||(B-1).*W||_inf, ||B.*W||_inf (max absolute row sums; rows are
    output channels) for bf16 weights [C_out, ...] and one 2:4 pattern per group."""
    _need_cuda(w, pattern, out)
    c_out = w.shape[0]
    k = w.numel() // c_out
    if out is None:
        out = torch.empty((3,), dtype=torch.float32, device=w.device)
    f = lib().ssconv_mask_norms
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
    _check("ssconv_mask_norms", f(_ptr(w), _ptr(pattern), c_out, k, _ptr(out), _stream(stream)))
    return out


def ssconv_absmax(x: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """fp32 [1] on the device: the largest magnitude in a bf16 tensor."""
    _need_cuda(x, out)
    if out is None:
        out = torch.empty((1,), dtype=torch.float32, device=x.device)
    f = lib().ssconv_absmax
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
    _check("ssconv_absmax", f(_ptr(x), x.numel(), _ptr(out), _stream(stream)))
    return out


def ssconv_stability_threshold(lemma: int, L: float, layer_norms, j: int, extra_norm: float, x_norm: float) -> float:
    """Confidence threshold of Lemma 3.4 / 3.5 / 3.6 (host arithmetic in the library)."""
    n = len(layer_norms)
    arr = (ctypes.c_double * n)(*[float(v) for v in layer_norms])
    f = lib().ssconv_stability_threshold
    f.restype = ctypes.c_double
    f.argtypes = [ctypes.c_int32, ctypes.c_double, ctypes.POINTER(ctypes.c_double), ctypes.c_int32, ctypes.c_int32,
                  ctypes.c_double, ctypes.c_double]
    v = float(f(lemma, float(L), arr, n, j, float(extra_norm), float(x_norm)))
    if v < 0:
        raise ValueError("bad arguments to ssconv_stability_threshold")
    return v


def ssconv_dgrad_prepare(desc: Desc, w: Optional[torch.Tensor], stream=None):
    """(desc_dx, w_t) for the input gradient of a layer: dx = ssconv_forward_dense(desc_dx, dy, w_t), with dy
    passed through ssconv_dgrad_spread first when the layer's stride is above 1.
    w_t bf16 [C_in,KH,KW,C_out] holds the reversed, channel-exchanged filter (None if w is None)."""
    _need_cuda(w)
    out = Desc()
    w_t = None
    if w is not None:
        w_t = torch.empty((desc.C_in, desc.KH, desc.KW, desc.C_out), dtype=torch.bfloat16, device=w.device)
    f = lib().ssconv_dgrad_prepare
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(Desc), ctypes.c_void_p]
    _check("ssconv_dgrad_prepare", f(ctypes.byref(desc), _ptr(w), _ptr(w_t), ctypes.byref(out), _stream(stream)))
    return out, w_t


def ssconv_dgrad_spread(desc: Desc, dy: torch.Tensor, stream=None) -> torch.Tensor:
    """dy [N,H_out,W_out,C_out] of a strided layer spread out with zeros to [N,Hz,Wz,C_out],
    Hz = H + 2 pad - dil (KH - 1): the input of the convolution ssconv_dgrad_prepare describes."""
    _need_cuda(dy)
    Hz = ssconv_window_extent(desc.H, desc.KH, 1, desc.pad_h, desc.dil_h)   # all unit-stride filter placements
    Wz = ssconv_window_extent(desc.W, desc.KW, 1, desc.pad_w, desc.dil_w)
    out = torch.empty((desc.N, Hz, Wz, desc.C_out), dtype=torch.bfloat16, device=dy.device)
    f = lib().ssconv_dgrad_spread
    f.restype = ctypes.c_int32
    f.argtypes = [ctypes.POINTER(Desc), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    _check("ssconv_dgrad_spread", f(ctypes.byref(desc), _ptr(dy), _ptr(out), _stream(stream)))
    return out
