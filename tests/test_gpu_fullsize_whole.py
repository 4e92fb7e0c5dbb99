"""Every output element of whole layer passes at the benchmark sizes, through the
schedule the benchmark times (two streams, then the same pass replayed from a
CUDA graph), against the oracle run on the copied-back 16-bit inputs.

The oracle needs a few seconds per input on a many-core host, so nothing is
sampled here: every channel's statistics and factors, every code, Step,
zero-point and corrected bias of every matrix, and (W8A8) every activation code
are compared.  The oracle's results for an input are computed once and serve
both the eager two-stream pass and the graph replay (and both weight
bit-widths of the group-quantised layer).
"""
import numpy as np
import pytest
import torch

from oracle import aweq_oracle as orc
from paper_2311_01305_b200 import synth
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _dt(wl):
    return orc.F16 if wl.dtype == "f16" else orc.BF16


def _mean_abs(X: torch.Tensor) -> np.ndarray:
    """mean |x| per channel, only used as the floor of the tolerance of the mean."""
    acc = torch.zeros(X.shape[1], dtype=torch.float64, device=X.device)
    for r0 in range(0, X.shape[0], 16384):
        acc += X[r0:r0 + 16384].abs().double().sum(dim=0)
    return (acc / X.shape[0]).cpu().numpy()


def _scramble(cal):
    for group in cal.out.values():
        for t in group.values():
            t.view(torch.uint8).fill_(0xA5)


def _oracle_input_side(wl, inp, X, W):
    """Steps 1-3 of one input (and step 6 for W8A8) on the host copy of its bits."""
    lins = [l for l in wl.linears if l.input == inp.name]
    xb = util.bits(X[inp.name])
    xs = orc.stats(xb, _dt(wl))
    wr = None
    for l in lins:
        wr = orc.wrange(util.bits(W[l.name]), _dt(wl), prev=wr)
    f = orc.factors(xs[0], xs[1], xs[2], wr[0], wr[1])
    ref = {"stats": xs, "wrange": wr, "factors": f, "mean_abs": _mean_abs(X[inp.name])}
    if wl.act_quant:
        ref["act"] = orc.quant_act(xb, _dt(wl), f["rinv"], orc.PER_ROW)
    return ref


def _oracle_weights(wl, inp, W, f, bits):
    gran = orc.PER_ROW if wl.w_gran == "row" else orc.PER_GROUP
    out = {}
    for l in (l for l in wl.linears if l.input == inp.name):
        codes, step, zp, delta = orc.equalize_quantize(util.bits(W[l.name]), _dt(wl), f["s"], f["mu_hat"], bits, gran,
                                                       wl.group)
        bf, b16 = orc.bias_correct(delta, None, _dt(wl))
        out[l.name] = {"codes": codes, "step": step, "zp": zp, "bias_f32": bf, "bias_16": b16}
    return out


def _check_input(cal, inp, ref, with_act=True):
    o = cal.out[inp.name]
    got = {k: o[k].cpu().numpy() for k in ("xmin", "xmax", "xmean", "wmin", "wmax", "s", "rinv", "mu_hat", "pX", "pW",
                                           "scalars")}
    xs, wr, f = ref["stats"], ref["wrange"], ref["factors"]
    util.assert_same_values(got["xmin"], xs[0], inp.name + " xmin")
    util.assert_same_values(got["xmax"], xs[1], inp.name + " xmax")
    assert np.all(np.abs(got["xmean"].astype(np.float64) - xs[2]) <= util.mean_tolerance(xs[2], ref["mean_abs"]))
    util.assert_same_values(got["wmin"], wr[0], inp.name + " wmin")
    util.assert_same_values(got["wmax"], wr[1], inp.name + " wmax")
    util.assert_same_values(got["s"], f["s"], inp.name + " s")
    util.assert_same_values(got["rinv"], f["rinv"], inp.name + " 1/s")
    assert np.allclose(got["mu_hat"], f["mu_hat"], rtol=1e-6, atol=1e-9 * ref["mean_abs"].max())
    assert np.allclose(got["pX"], f["pX"], rtol=1e-6) and np.allclose(got["pW"], f["pW"], rtol=1e-6)
    assert np.allclose(got["scalars"], f["scalars"], rtol=1e-6)
    if with_act and "act" in ref:
        xq, st, z = ref["act"]
        util.assert_same_values(o["act_zp"].cpu().numpy(), z, inp.name + " act zp")
        util.assert_same_values(o["act_step"].cpu().numpy(), st, inp.name + " act step")
        dev_ref = torch.from_numpy(xq).to(DEV)
        assert torch.equal(o["Xq"], dev_ref), inp.name + " activation codes"
        del dev_ref


def _check_weights(cal, wref, dtype_tag):
    for name, r in wref.items():
        lo = cal.out[name]
        util.assert_same_values(lo["zp"].cpu().numpy(), r["zp"], name + " zp")
        util.assert_same_values(lo["step"].cpu().numpy(), r["step"], name + " step")
        util.assert_same_values(lo["codes"].cpu().numpy(), r["codes"], name + " codes")
        b32 = lo["bias_f32"].cpu().numpy()
        assert np.allclose(b32, r["bias_f32"], rtol=0, atol=1e-5), name
        # the 16-bit bias is the library's own binary32 bias rounded once
        util.assert_same_values(util.bits(lo["bias"]), orc.encode16(b32, dtype_tag), name + " bias16")


def _whole_layer(name, bits_list):
    from paper_2311_01305_b200 import aweq, calibrate
    wl = synth.workloads()[name]
    X, W = synth.generate(wl, DEV)
    refs = {inp.name: _oracle_input_side(wl, inp, X, W) for inp in wl.inputs}
    for bits in bits_list:
        wrefs = {inp.name: _oracle_weights(wl, inp, W, refs[inp.name]["factors"], bits) for inp in wl.inputs}
        cal = calibrate.LayerCalibrator(wl, bits, X, W, None, overlap=True)
        assert cal.overlap
        _scramble(cal)
        cal.run()                                            # two streams, eager
        torch.cuda.synchronize()
        assert aweq.read_status(cal.status) == {"nonfinite": 0, "zero_range": 0, "wait_timeout": 0}
        for inp in wl.inputs:
            _check_input(cal, inp, refs[inp.name])
            _check_weights(cal, wrefs[inp.name], _dt(wl))
        graph = cal.capture()                                # the same pass as one graph launch
        _scramble(cal)
        graph.replay()
        torch.cuda.synchronize()
        assert aweq.read_status(cal.status)["wait_timeout"] == 0
        for inp in wl.inputs:
            _check_input(cal, inp, refs[inp.name])
            _check_weights(cal, wrefs[inp.name], _dt(wl))
        del cal, graph
        torch.cuda.empty_cache()


def test_llama7b_layer_w4_and_w3_every_element():
    _whole_layer("llama7b_layer_w4w3_g128", (4, 3))


def test_opt125m_model_layer_w8a8_every_element():
    _whole_layer("opt125m_model_w8a8", (8,))


def test_llama13b_layer_w8a8_every_element():
    _whole_layer("llama13b_layer_w8a8", (8,))
