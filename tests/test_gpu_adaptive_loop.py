"""Alg. 1 on a small stack of linear layers: every F steps the probe measures V_s, V_act, V_w per
layer and the ratio update moves (s, rho_l, nu_l); the trajectory computed with the CUDA library must
be the one the oracle computes from the same inputs."""
import numpy as np
import pytest
import torch

from oracle import vcas_oracle as o
from paper_2402_17227_b200 import binding as vb
from paper_2402_17227_b200 import build as vbuild
from paper_2402_17227_b200 import inputs
from tests.util import f32, np64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,path", [(torch.float32, vb.GEMM_FMA), (torch.bfloat16, vb.GEMM_TENSOR)])
def test_adaptive_ratio_trajectory_matches_oracle(dtype, path):
    vbuild.build()
    N, T, M, periods = 8, 16, 2, 5
    shapes = [(64, 128), (128, 64), (64, 64)]                 # (d_in, d_out) of layers 1..3
    cfg = vb.default_config()
    cfg.M = M
    cfg.alpha, cfg.beta, cfg.tau_act, cfg.tau_w = 0.05, 0.8, 0.5, 0.5     # coarse steps: visible movement
    cases = [inputs.LayerCase(f"l{i}", N, T, di, do, dtype, 1.5, 1.0, 1.0, 1.0, data_seed=100 + i)
             for i, (di, do) in enumerate(shapes)]
    layers = [vb.Layer(N, T, di, do, dtype, path, cfg) for di, do in shapes]
    L = len(layers)
    kw = dict(tau_act=f32(0.5), tau_w=f32(0.5), alpha=f32(0.05), beta=f32(0.8))
    s_g, rho_g, nu_g = 1.0, [1.0] * L, [1.0] * L              # library state
    s_o, rho_o, nu_o = 1.0, np.ones(L), np.ones(L)            # oracle state
    moved = False
    for period in range(periods):
        Vg = np.zeros((L, 5)); Vo = np.zeros((L, 5))
        for l in range(L):
            batches = [inputs.make_layer(cases[l], batch=period * M + i) for i in range(M)]
            W = batches[0][2]
            out = layers[l].variance_probe([b[0].cuda() for b in batches], [b[1].cuda() for b in batches], W.cuda(),
                                           float(rho_g[l]), float(nu_g[l]), float(s_g), 1000 * period + l)
            Vg[l] = out.cpu().numpy()
            ref = o.variance_probe([np64(b[0]) for b in batches], [np64(b[1]) for b in batches], np64(W), N, T,
                                   f32(rho_o[l]), f32(nu_o[l]), s=f32(s_o), alpha=f32(0.05), seed=1000 * period + l)
            Vo[l] = [ref["V_s"], ref["V_act"], ref["V_w"], ref["p_lo"], ref["p_hi"]]
        tol = 1e-3 if dtype == torch.float32 else 3e-2
        assert np.allclose(Vg[:, :3], Vo[:, :3], rtol=tol, atol=1e-12), (period, Vg, Vo)
        assert np.allclose(Vg[:, 3:], Vo[:, 3:], atol=1e-6)
        s_g, rho_g, nu_g = vb.update_ratios(s_g, rho_g, nu_g, Vg[:, 0], Vg[:, 1], Vg[:, 2], Vg[:, 3], Vg[:, 4], cfg)
        s_o, rho_o, nu_o = o.update_ratios(s_o, rho_o, nu_o, Vo[:, 0], Vo[:, 1], Vo[:, 2], Vo[:, 3], Vo[:, 4], **kw)
        assert s_g == pytest.approx(s_o, abs=1e-6)
        assert np.allclose(rho_g, rho_o, atol=1e-6) and np.allclose(nu_g, nu_o, rtol=1e-5)
        assert np.all(np.diff(rho_g) >= 0) and 0.0 <= s_g <= 1.0 and max(nu_g) <= 1.0
        moved = moved or s_g < 1.0 or min(nu_g) < 1.0
        # F backward steps at the current ratios would follow here; one per layer keeps the test short
        for l in range(L):
            X, dY, W = [t.cuda() for t in inputs.make_layer(cases[l], batch=77 + period)]
            layers[l].linear_bwd(X, dY, W, max(float(rho_g[l]), 1e-3), float(nu_g[l]), period)
            assert layers[l].device_status() == 0
    assert moved                                              # the ratios did adapt
    for lay in layers:
        lay.close()
