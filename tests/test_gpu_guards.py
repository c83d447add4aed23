"""Memory-safety nets that stand in for a sanitizer: guard bands and the bounded wait.

Guard bands: outputs and scratch buffers are carved out of larger allocations whose slack on both
sides holds a sentinel pattern; after the calls the slack must be untouched.  Covered: the output of
the one-block kernel (TMA stores, ragged channels and positions), of the K-split path (finishing
kernel), of the pair kernel (tests/test_gpu_pair.py), the forward workspace and the weight gradient's
scratch and output.

Bounded wait: every mbarrier wait in the library gives up after a cycle limit, raises a flag and lets
the kernel return with SSCONV_ERR_TIMEOUT in the caller's status word.  No product kernel is broken to
show it; a one-block self-test kernel of the library waits on a barrier nobody arrives at.
"""
import time

import pytest
import torch

from paper_2411_00288_b200 import api, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
BAND = 1 << 16  # bytes of slack on each side


def _banded(nbytes, fill=0x5A):
    """(whole buffer uint8, view of the middle `nbytes`); the middle starts 256-byte aligned."""
    buf = torch.full((nbytes + 2 * BAND,), fill, dtype=torch.uint8, device=DEV)
    return buf, buf[BAND:BAND + nbytes]


def _bands_intact(buf, nbytes, fill=0x5A):
    return bool((buf[:BAND] == fill).all()) and bool((buf[BAND + nbytes:] == fill).all())


@pytest.mark.parametrize("case", [
    ("guard_ragged", 3, 13, 11, 64, 72, 3, 1, 1),       # ragged channels and positions, whole tiles
    ("guard_split", 8, 7, 7, 512, 264, 3, 1, 1),        # K split: partial tiles parked in ws, finishing kernel
    ("guard_1x1_s2", 2, 15, 15, 64, 136, 1, 2, 0),      # strided 1x1
], ids=lambda c: c[0])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_forward_touches_neither_the_slack_around_y_nor_around_ws(case, sparse):
    name, n, h, w, ci, co, k, s, p = case
    spec = synth.LayerSpec(name, n, h, w, ci, co, k, k, s, p, 1, relu=True, w_std="fan_in", mask_source="magnitude",
                           config=11, index={"guard_ragged": 1, "guard_split": 2, "guard_1x1_s2": 3}[name])
    inp = synth.make_inputs(spec)
    desc = api.desc_from_spec(spec)
    wd, bias = inp.w.to(DEV), inp.bias.to(DEV)
    n_out = spec.P * spec.C_out * 2
    ybuf, ymid = _banded(n_out)
    y = ymid.view(torch.bfloat16).view(spec.N, spec.H_out, spec.W_out, spec.C_out)
    ws_bytes = api.ssconv_sizes(desc).ws_bytes_sparse
    wsbuf, ws = _banded(ws_bytes)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    if sparse:
        pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, wd, spec.G)
        w_comp, meta = api.ssconv_compress(desc, wd, pat)
        api.ssconv_forward(desc, inp.x.to(DEV), w_comp, meta, bias, y=y, ws=ws, dev_status=status)
    else:
        api.ssconv_forward_dense(desc, inp.x.to(DEV), wd, bias, y=y, ws=ws, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert _bands_intact(ybuf, n_out), "the slack around y was written"
    assert _bands_intact(wsbuf, ws_bytes), "the slack around ws was written"
    assert bool((y >= 0).all()), "ReLU output: every element must have been written"
    if name == "guard_split":
        assert api.ssconv_plan(desc, sparse)["split"]
        assert bool((ws != 0x5A).any()), "the split path parks partial tiles in ws"


def test_weight_gradient_touches_neither_the_slack_around_dw_nor_around_its_scratch():
    spec = synth.LayerSpec("guard_wgrad", 4, 14, 14, 72, 136, 3, 3, 1, 1, 1, config=11, index=60)
    inp = synth.make_inputs(spec, x_only=True)
    tr = synth.make_train_inputs(spec)
    desc = api.desc_from_spec(spec)
    n_dw = spec.C_out * spec.K * 4
    dwbuf, dwmid = _banded(n_dw)
    dw = dwmid.view(torch.float32).view(spec.C_out, spec.KH, spec.KW, spec.C_in)
    need = api.ssconv_wgrad_ws_bytes(desc)
    wsbuf, ws = _banded(max(need, 256))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.ssconv_wgrad(desc, inp.x.to(DEV), tr.dy.to(DEV), dw=dw, ws=ws, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert _bands_intact(dwbuf, n_dw) and _bands_intact(wsbuf, max(need, 256))
    assert bool(torch.isfinite(dw).all())


def test_bounded_wait_runs_out_returns_a_status_and_leaves_the_context_usable():
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    t0 = time.perf_counter()
    api.ssconv_selftest_wait_timeout(200_000, status)      # 0.1 ms of SM clock
    torch.cuda.synchronize()                               # returns: the kernel gave up by itself
    assert time.perf_counter() - t0 < 5.0
    assert int(status.item()) == api.ERR_TIMEOUT
    assert "timed out" in api.status_string(int(status.item()))
    # the device and the library work as before
    spec = synth.config_layers(1)[0]
    rel, mx = parity.check_layer(spec, DEV, sparse=True)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL
    with pytest.raises(api.SsconvError):
        api.ssconv_selftest_wait_timeout(10, status)       # limit below the accepted range


def test_calls_on_two_streams_with_their_own_scratch_do_not_disturb_each_other():
    """The library keeps no hidden device state between calls (the one entry point that does says so in the
    header): two layers launched again and again on two streams that overlap on the GPU, each with its own
    scratch and status word, give bit for bit what they give alone.  A K-split layer (scratch + finishing
    kernel) on one stream, a layer for the thread-block-pair kernel on the other."""
    specs = [synth.LayerSpec("deep_k_split", 2, 7, 7, 512, 128, 3, 3, 1, 1, 1, config=14, index=0),
             synth.LayerSpec("pair_3x3", 8, 14, 14, 256, 256, 3, 3, 1, 1, 1, config=14, index=1)]
    ctx = []
    for spec in specs:
        inp = synth.make_inputs(spec)
        desc = api.desc_from_spec(spec)
        w = inp.w.to(DEV)
        pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
        w_comp, meta = api.ssconv_compress(desc, w, pat)
        ws = torch.empty((api.ssconv_sizes(desc).ws_bytes_sparse,), dtype=torch.uint8, device=DEV)
        ctx.append(dict(desc=desc, x=inp.x.to(DEV), w_comp=w_comp, meta=meta, bias=inp.bias.to(DEV), ws=ws,
                        status=torch.zeros(1, dtype=torch.int32, device=DEV), stream=torch.cuda.Stream(device=DEV)))
    torch.cuda.synchronize()

    def run(c, y):
        api.ssconv_forward(c["desc"], c["x"], c["w_comp"], c["meta"], c["bias"], y=y, ws=c["ws"], dev_status=c["status"],
                           stream=c["stream"])

    alone = []
    for c in ctx:
        y = torch.empty((c["desc"].N, *api.ssconv_out_shape(c["desc"]), c["desc"].C_out), dtype=torch.bfloat16, device=DEV)
        run(c, y)
        torch.cuda.synchronize()
        alone.append(y.clone())
    outs = [[torch.empty_like(a) for _ in range(12)] for a in alone]
    for it in range(12):
        for c, o in zip(ctx, outs):
            run(c, o[it])
    torch.cuda.synchronize()
    for c, a, o in zip(ctx, alone, outs):
        assert int(c["status"].item()) == 0
        for y in o:
            assert torch.equal(y, a)
