"""Helpers shared by the GPU parity tests: run one layer through the CUDA library (via the
C ABI binding) and through the CPU oracle on the same seeded bits, and compare."""
import dataclasses
import math

import numpy as np
import torch

from oracle import masks
from oracle.conv import ConvShape, conv2d_f64, conv2d_f64_sample
from paper_2411_00288_b200 import api, synth

# spec gates for convolution outputs
REL_FRO_TOL = 5e-3
MAX_ABS_TOL = 2e-2


def oracle_shape(spec) -> ConvShape:
    return ConvShape(spec.N, spec.H, spec.W, spec.C_in, spec.C_out, spec.KH, spec.KW,
                     (spec.stride, spec.stride), (spec.pad, spec.pad), (spec.dil, spec.dil),
                     relu=spec.relu and not spec.gelu)


def oracle_pattern(inp) -> np.ndarray:
    """Pattern per group from the oracle, by the layer's mask source."""
    spec = inp.spec
    if spec.mask_source == "magnitude":
        return masks.select_from_magnitude(synth.bf16_bits(inp.w))
    if spec.mask_source == "gumbel_logits":
        return masks.select_from_logits(inp.scores.numpy())
    return inp.pattern.numpy().astype(np.uint8)


def gpu_pattern(inp, dev) -> torch.Tensor:
    """Pattern per group from the CUDA library (or the given one for uniform_pattern)."""
    spec = inp.spec
    if spec.mask_source == "magnitude":
        return api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, inp.w.to(dev), spec.G)
    if spec.mask_source == "gumbel_logits":
        return api.ssconv_select_mask(api.MASK_LOGITS_F32, inp.scores.to(dev), spec.G)
    return inp.pattern.to(dev)


def bf16_tensor_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float32).numpy().astype(np.float64)


def gelu_f64(x: np.ndarray) -> np.ndarray:
    """GELU in its defining form x * Phi(x), Phi the standard normal distribution function."""
    erf = np.vectorize(math.erf, otypes=[np.float64])
    return 0.5 * x * (1.0 + erf(x / math.sqrt(2.0)))


def errors(y_gpu_f64: np.ndarray, y_ref: np.ndarray):
    diff = y_gpu_f64 - y_ref
    denom = np.linalg.norm(y_ref.reshape(-1))
    rel = float(np.linalg.norm(diff.reshape(-1)) / denom) if denom > 0 else float(np.abs(diff).max())
    return rel, float(np.abs(diff).max())


def run_layer_gpu(inp, dev, sparse=True, pattern=None, residual=None):
    """Returns (y bf16 on device, dev_status int).  Dense path uses the raw (unmasked) weights
    unless `pattern` is given, in which case it gets the masked weights from decompress."""
    spec = inp.spec
    desc = api.desc_from_spec(spec)
    x = inp.x.to(dev)
    w = inp.w.to(dev)
    bias = inp.bias.to(dev) if inp.bias is not None else None
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    if sparse:
        pat = gpu_pattern(inp, dev) if pattern is None else pattern
        w_comp, meta = api.ssconv_compress(desc, w, pat)
        y = api.ssconv_forward(desc, x, w_comp, meta, bias, dev_status=status, residual=residual)
    else:
        y = api.ssconv_forward_dense(desc, x, w, bias, dev_status=status, residual=residual)
    torch.cuda.synchronize()
    return y, int(status.item())


def make_residual(spec, seed=None) -> torch.Tensor:
    """Seeded bf16 tensor of the layer's output shape (its own stream of the layer's seed)."""
    g = torch.Generator().manual_seed((spec.seed if seed is None else seed) + 90_000_000)
    return torch.randn((spec.N, spec.H_out, spec.W_out, spec.C_out), generator=g, dtype=torch.float32).to(torch.bfloat16)


def check_layer(spec, dev, sparse=True, sample=None, seed=None, residual=False):
    """Full (or sampled) parity of one layer against the oracle; returns (rel_fro, max_abs).
    With residual=True the fused call y = act(bias + conv + residual) is checked: the oracle computes
    the convolution without activation, the test adds the residual and applies the activation in fp64."""
    inp = synth.make_inputs(spec, seed=seed)
    res = make_residual(spec, seed) if residual else None
    y, st = run_layer_gpu(inp, dev, sparse=sparse, residual=res.to(dev) if residual else None)
    assert st == 0, f"device status {st}"
    pat = oracle_pattern(inp)
    w_bits = synth.bf16_bits(inp.w)
    mask = masks.mask_from_pattern(pat, w_bits.shape) if sparse else None
    bias = inp.bias.numpy() if inp.bias is not None else None
    shp = oracle_shape(spec)
    if residual or spec.gelu:
        shp = dataclasses.replace(shp, relu=False)  # the test finishes the epilogue in fp64 itself
    yg = bf16_tensor_to_f64(y)

    def finish(ref, idx=None):
        if not residual and not spec.gelu:
            return ref
        if residual:
            r = bf16_tensor_to_f64(res).reshape(-1)
            ref = ref + (r.reshape(ref.shape) if idx is None else r[idx])
        if spec.gelu:
            return gelu_f64(ref)
        return np.maximum(ref, 0.0) if spec.relu else ref

    if sample is None:
        ref = finish(conv2d_f64(shp, synth.bf16_bits(inp.x), w_bits, mask=mask, bias=bias))
        assert ref.shape == yg.shape
        return errors(yg, ref)
    rng = np.random.default_rng(spec.seed & 0xFFFFFFFF)
    idx = rng.choice(yg.size, size=min(sample, yg.size), replace=False)
    ref = finish(conv2d_f64_sample(shp, synth.bf16_bits(inp.x), w_bits, idx, mask=mask, bias=bias), idx)
    return errors(yg.reshape(-1)[idx], ref)
