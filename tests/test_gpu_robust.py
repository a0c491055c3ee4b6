"""GPU parity on inputs that stress the numerical decisions of the expert kernels rather than their indexing:
activations with a large mean (the reason the kernels convert the codes exactly by default: the optional
offset-subnormal conversion of the tcgen05 up/gate kernel subtracts 128 * sum(x)), and expert weights whose row scales spread over orders
of magnitude (the fp16 intermediate of the down projection is placed by the expert's largest row scale). The bar is
the same as everywhere: 2e-3 in the pre-rounding measure, against the oracle, through both kernel families."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_38090_b200 import inputs
from gpu_util import Workload, gate_a, gate_b, gate_c

pytestmark = pytest.mark.gpu
TOL = 2e-3


def _run(wl, sh, T, fmt=0, conversion=0, force=False, fp32=True, layout=0):
    from paper_2609_38090_b200 import binding as b
    d = wl.device_inputs()
    m = b.Mira(sh.C, sh.R, sh.E, n_shared=sh.n_shared, n_layers=4, max_tokens=T, max_top_k=sh.k, out_fp32=fp32, fmt=fmt)
    blobs = m.quantize_experts(d["w1"], d["w2"], d["w3"])
    assert np.array_equal(blobs.cpu().numpy(), np.stack(wl.blobs))
    m.up_conversion(conversion)
    m.force_decode_path(force)
    m.tensor_layout(layout)
    slot_map = torch.arange(sh.E + sh.n_shared, dtype=torch.int32, device="cuda")
    out = m.moe_layer(d["x"], d["wr"], d["bias"], b.slot_table(blobs), slot_map, sh.k)
    torch.cuda.synchronize()
    assert m.poll_status()[0] == 0
    return out


def _shifted(sh, T, mu, spread=0.1):
    g = np.random.default_rng(5)
    x = mu + spread * g.standard_normal((T, sh.C))
    x[0] = np.abs(x[0]) + 0.5                      # one row with no negative entry at all
    return inputs.round_to_bf16(x.astype(np.float32))


@pytest.mark.parametrize("T", [8, 80])             # the weight-streaming kernels and the tcgen05 kernels
@pytest.mark.parametrize("C,mu", [(4096, 0.1), (4096, 1.0), (16384, 0.03), (16384, 1.0), (1024, 1.0)])
def test_activations_with_a_large_mean(C, mu, T):
    sh = inputs.LayerShape("dc", C=C, R=256, E=4, k=2, T=T, seed=21)
    wl = Workload(sh, T)
    wl.x = _shifted(sh, T, mu)
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k)
    out = _run(wl, sh, T)
    assert gate_a(out.cpu().numpy(), res["out64"]) <= TOL
    out_bf16 = _run(wl, sh, T, fp32=False).float().cpu().numpy()
    assert gate_b(out_bf16, res["out64"]) <= TOL and gate_c(out_bf16, res["out64"], bf16_output=True) <= TOL
    assert torch.equal(out, _run(wl, sh, T, conversion=1))        # the default IS the exact conversion


def test_offset_conversion_is_an_option_for_zero_mean_batches():
    """MIRA_OPT_UP_CONVERSION = 2 (the tcgen05 up/gate kernel's cheaper offset form) holds the tolerance on the
    synthetic zero-mean workload and fails it on a shifted one, which is why it is not the default."""
    T = 80
    sh = inputs.LayerShape("zm", C=4096, R=256, E=4, k=2, T=T, seed=22)
    wl = Workload(sh, T)
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k)
    auto, exact, offset = (_run(wl, sh, T, conversion=c) for c in (0, 1, 2))
    assert torch.equal(auto, exact)
    for out in (exact, offset):
        assert gate_a(out.cpu().numpy(), res["out64"]) <= TOL
    wl.x = _shifted(sh, T, 1.0)
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k)
    assert gate_a(_run(wl, sh, T).cpu().numpy(), res["out64"]) <= TOL
    assert gate_a(_run(wl, sh, T, conversion=2).cpu().numpy(), res["out64"]) > TOL


def _lognormal_rows(shape, e):
    """Row scales spread log-normally (sigma 1.5: a factor of about 400 between the smallest and the largest of a
    few hundred rows), applied to the up and the gate row alike."""
    w1, w2, w3 = inputs.expert_weights(shape, e)
    s = np.exp(1.5 * np.random.default_rng(100 + e).standard_normal((shape.R, 1))).astype(np.float32)
    return w1 * s, w2, w3 * s


@pytest.mark.parametrize("fmt", [0, 1])
@pytest.mark.parametrize("T,force", [(8, False), (80, False), (80, True)])
@pytest.mark.parametrize("shape", ["tiny", "wide"])
def test_log_normal_row_scales(shape, T, force, fmt):
    sh = inputs.TINY if shape == "tiny" else inputs.LayerShape("h2", C=1024, R=2048, E=4, k=2, T=T, seed=4)
    wl = Workload(sh, T, gen=_lognormal_rows, fmt=fmt)
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k, fmt=fmt)
    out = _run(wl, sh, T, fmt=fmt, force=force).cpu().numpy()
    assert np.isfinite(out).all() and gate_a(out, res["out64"]) <= TOL


def _outlier_rows(shape, e):
    """The quantizer test's heavy recipe: up-projection rows scaled log-normally (sigma 2) with the gate rows left
    alone, and one down-projection weight in a hundred nine times larger. In the shared format a row's scale then
    follows its up row, the gate and down codes of the large rows shrink towards zero, and the rows that carry the
    output are far smaller than the largest scale suggests."""
    w1, w2, w3 = inputs.expert_weights(shape, e)
    g = np.random.default_rng(100 + e)
    w1 = w1 * np.exp(2 * g.standard_normal((shape.R, 1))).astype(np.float32)
    w2[g.random(w2.shape) < 0.01] *= np.float32(9.0)
    return w1, w2, w3


def _outliers_in_two_experts(shape, e):
    return _outlier_rows(shape, e) if e in (1, 2) else inputs.expert_weights(shape, e)


@pytest.mark.parametrize("fmt", [0, 1])
@pytest.mark.parametrize("T,force", [(8, False), (80, False), (80, True), (300, False)])
@pytest.mark.parametrize("shape,gen", [("tiny", _outlier_rows), ("wide", _outlier_rows), ("tiny", _outliers_in_two_experts)])
def test_outlier_rows_take_the_two_window_intermediate(shape, gen, T, force, fmt):
    """Experts whose row scales spread over more than a factor of 8 keep their fp16 intermediate in two windows
    (2^24 apart) and run the down projection over both; the others, in the same batch, stay on one."""
    sh = inputs.TINY if shape == "tiny" else inputs.LayerShape("h2", C=1024, R=2048, E=4, k=2, T=T, seed=4)
    wl = Workload(sh, T, gen=gen, fmt=fmt)
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k, fmt=fmt)
    out = _run(wl, sh, T, fmt=fmt, force=force).cpu().numpy()
    assert np.isfinite(out).all() and gate_a(out, res["out64"]) <= TOL
    out_bf16 = _run(wl, sh, T, fmt=fmt, force=force, fp32=False).float().cpu().numpy()
    assert gate_b(out_bf16, res["out64"]) <= TOL and gate_c(out_bf16, res["out64"], bf16_output=True) <= TOL


@pytest.mark.parametrize("fmt", [0, 1])
@pytest.mark.parametrize("layout", [4, 5])
def test_outlier_rows_on_the_two_sm_kernel(layout, fmt):
    """The two windows of a wide-range expert on the cta_group::2 kernel: the leader CTA holds the upper window of a
    tile's tokens, its peer the lower one."""
    sh = inputs.TINY
    for T in (80, 300):
        wl = Workload(sh, T, gen=_outliers_in_two_experts, fmt=fmt)
        res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k, fmt=fmt)
        out = _run(wl, sh, T, fmt=fmt, layout=layout).cpu().numpy()
        assert np.isfinite(out).all() and gate_a(out, res["out64"]) <= TOL
