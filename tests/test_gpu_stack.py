"""The ResNet-50-shaped convolution stack (stem, max-pool, 52 masked convolutions) run end to end on
the GPU, checked layer by layer against the fp64 oracle.

The check is teacher-forced: every layer's oracle receives the bf16 input that the GPU layer before
it actually produced, so errors do not compound over the 53 convolutions and each layer meets the
same gates as a stand-alone layer."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import masks
from oracle.conv import conv2d_f64, conv2d_f64_sample
from paper_2411_00288_b200 import api, stack, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _stack_input(n, seed=77):
    g = torch.Generator().manual_seed(synth.SEED_BASE + 500 + seed)
    x = torch.zeros((n, 224, 224, 8), dtype=torch.bfloat16)
    x[..., :3] = torch.randn((n, 224, 224, 3), generator=g, dtype=torch.float32).to(torch.bfloat16)
    return x  # channels 3..7 are the zero padding of the 3-channel image


def _maxpool_reference(x):
    """3x3 stride-2 pad-1 max over an NHWC float array (padding never wins: -inf)."""
    n, h, w, c = x.shape
    ho, wo = (h - 1) // 2 + 1, (w - 1) // 2 + 1
    xp = np.full((n, h + 2, w + 2, c), -np.inf, dtype=x.dtype)
    xp[:, 1:-1, 1:-1] = x
    out = np.full((n, ho, wo, c), -np.inf, dtype=x.dtype)
    for kh in range(3):
        for kw in range(3):
            out = np.maximum(out, xp[:, kh:kh + 2 * ho:2, kw:kw + 2 * wo:2])
    return out


def _check_stack(n, sample, residual=False, raw_images=False):
    """raw_images: hand the stack the 3-channel images (its stem then runs through space-to-depth)
    instead of images already padded to 8 channels (width unfold); the oracle sees the padded form."""
    steps = synth.resnet50_stack(n, residual=residual)
    net = stack.ConvStack(steps, DEV)
    x = _stack_input(n)
    xd = x[..., :3].contiguous().to(DEV) if raw_images else x.to(DEV)
    c0 = api.ssconv_launch_count()
    net.forward(xd, sparse=True)
    torch.cuda.synchronize()
    assert api.ssconv_launch_count() - c0 >= 53
    assert int(net.status.item()) == 0
    worst = (0.0, 0.0, "")
    peak = 0.0
    for i, st in enumerate(steps):
        src = x if st.src < 0 else net.outputs[st.src].cpu()
        y = net.outputs[i].cpu()
        if st.kind == "maxpool":
            ref = _maxpool_reference(src.float().numpy())
            assert np.array_equal(y.float().numpy(), ref), "max-pool"
            continue
        spec = st.spec
        L = net.layers[i]
        w_bits = synth.bf16_bits(L["w_host"])
        mask = None
        if st.kind == "conv":
            pat = masks.select_from_magnitude(w_bits)
            assert np.array_equal(pat, L["pattern"].cpu().numpy()), f"{spec.name}: pattern"
            mask = masks.mask_from_pattern(pat, w_bits.shape)
        bias = L["bias_host"].numpy() if L["bias_host"] is not None else None
        shp = parity.oracle_shape(spec)
        res = net.outputs[st.res].cpu() if st.res >= 0 else None
        if res is not None:
            shp = dataclasses.replace(shp, relu=False)  # residual first, then the activation, in fp64 below
        if sample is None:
            yg = parity.bf16_tensor_to_f64(y)
            ref = conv2d_f64(shp, synth.bf16_bits(src), w_bits, mask=mask, bias=bias)
            if res is not None:
                ref = ref + parity.bf16_tensor_to_f64(res)
        else:
            rng = np.random.default_rng(spec.seed & 0xFFFFFFFF)
            idx = rng.choice(y.numel(), size=min(sample, y.numel()), replace=False)
            yg = parity.bf16_tensor_to_f64(y.reshape(-1)[torch.from_numpy(idx)])
            ref = conv2d_f64_sample(shp, synth.bf16_bits(src), w_bits, idx, mask=mask, bias=bias)
            if res is not None:
                ref = ref + parity.bf16_tensor_to_f64(res.reshape(-1)[torch.from_numpy(idx)])
        if res is not None and spec.relu:
            ref = np.maximum(ref, 0.0)
        rel, mx = parity.errors(yg, ref)
        assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{spec.name}: rel={rel:.3e} max={mx:.3e}"
        assert np.abs(yg).max() > 0, f"{spec.name}: all-zero output"
        if rel > worst[0]:
            worst = (rel, mx, spec.name)
        peak = max(peak, float(np.abs(yg).max()))
    print("largest |activation|", peak)
    return worst


def test_resnet50_stack_batch4_every_layer_full():
    worst = _check_stack(4, None)
    print("worst layer", worst)


def test_resnet50_stack_batch4_raw_images_every_layer_full():
    """The form the benchmark runs: 3-channel images in, the stem through space-to-depth."""
    worst = _check_stack(4, None, raw_images=True)
    print("worst layer", worst)


def test_resnet50_stack_batch256_raw_images_sampled():
    worst = _check_stack(256, 65536, raw_images=True)
    print("worst layer", worst)


def test_resnet50_stack_batch32_sampled():
    worst = _check_stack(32, 65536)
    print("worst layer", worst)


def test_resnet50_stack_with_skip_connections_batch4_full():
    """The same stack with the network's skip connections fused into the expand convolutions."""
    worst = _check_stack(4, None, residual=True)
    print("worst layer", worst)


def test_resnet50_stack_with_skip_connections_batch32_sampled():
    worst = _check_stack(32, 65536, residual=True)
    print("worst layer", worst)


def test_resnet50_stack_batch256_sampled():
    """The batch the end-to-end figure is quoted on; 65536 sampled outputs per layer."""
    worst = _check_stack(256, 65536)
    print("worst layer", worst)
