"""The probe on a sample of the parameters (App. D): the library picks the same rows of the parameter gradient
as the oracle's rule, and its V_s, V_act on those rows (scaled by d_out / rows) match the oracle's."""
import numpy as np
import pytest
import torch

from oracle import vcas_oracle as o
from paper_2402_17227_b200 import binding as vb
from paper_2402_17227_b200 import build as vbuild
from paper_2402_17227_b200 import inputs
from tests.util import f32, np64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,path,d_out,k", [(torch.bfloat16, vb.GEMM_TENSOR, 512, 128),
                                                (torch.bfloat16, vb.GEMM_TENSOR, 320, 64),
                                                (torch.float32, vb.GEMM_FMA, 136, 40)])
def test_probe_subsample_matches_oracle(dtype, path, d_out, k):
    vbuild.build()
    N, T, d_in, M = 8, 48, 128, 3
    case = inputs.LayerCase("ps", N, T, d_in, d_out, dtype, 1.0, 0.5, 0.5, 0.5)
    batches = [inputs.make_layer(case, batch=i) for i in range(M)]
    W = batches[0][2]
    cfg = vb.default_config()
    cfg.alpha = 0.05
    layer = vb.Layer(N, T, d_in, d_out, dtype, path, cfg)
    Xs, dYs = [b[0].cuda() for b in batches], [b[1].cuda() for b in batches]
    full = layer.variance_probe(Xs, dYs, W.cuda(), 0.5, 0.5, 0.75, 42).cpu().numpy()
    for sub_seed in (7, 2 ** 40 + 1):
        layer.set_probe_subsample(k, sub_seed)
        rows = layer.probe_subsample()
        assert rows == list(o.param_subset(d_out, k, sub_seed))                   # index work: exact
        out = layer.variance_probe(Xs, dYs, W.cuda(), 0.5, 0.5, 0.75, 42).cpu().numpy()
        ref = o.variance_probe([np64(b[0]) for b in batches], [np64(b[1]) for b in batches], np64(W), N, T, 0.5, 0.5,
                               s=0.75, alpha=f32(0.05), seed=42, param_rows=rows)
        tol = 1e-4 if dtype == torch.float32 else 2e-2
        assert out[0] == pytest.approx(ref["V_s"], rel=tol) and out[1] == pytest.approx(ref["V_act"], rel=tol)
        assert out[2] == pytest.approx(ref["V_w"], rel=1e-4) and out[2] == pytest.approx(full[2], rel=1e-6)
        assert out[3] == full[3] and out[4] == full[4]
        # an estimate of the full sums: same order of magnitude (k / d_out of the rows)
        assert 0.3 * full[0] < out[0] < 3 * full[0]
    layer.set_probe_subsample(0)
    again = layer.variance_probe(Xs, dYs, W.cuda(), 0.5, 0.5, 0.75, 42).cpu().numpy()
    assert np.array_equal(again, full)
    for bad in (k + 1, 512, d_out):
        with pytest.raises(vb.VcasError):
            layer.set_probe_subsample(bad, 1)
    assert layer.device_status() == 0
    layer.close()
