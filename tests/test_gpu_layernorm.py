"""SampleA in front of a LayerNorm (a layer that is not a matrix product): the CUDA backward against the oracle."""
import numpy as np
import pytest
import torch

from oracle import vcas_oracle as o
from paper_2402_17227_b200 import binding as vb
from paper_2402_17227_b200 import build as vbuild
from paper_2402_17227_b200 import inputs
from tests.util import f32, np64, rel_fro

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,tol", [(torch.bfloat16, 5e-3), (torch.float32, 1e-4)])
@pytest.mark.parametrize("N,T,d", [(6, 197, 320), (40, 33, 1024), (3, 130, 64)])
def test_layernorm_bwd_matches_oracle(dtype, tol, N, T, d):
    vbuild.build()
    case = inputs.LayerCase("ln", N, T, d, d, dtype, 1.5, 1.0, 0.5, 0.5)
    X, dY, _ = inputs.make_layer(case)
    X = (X.float() * 1.7 + 0.3).to(dtype)
    g = torch.Generator().manual_seed(5)
    gamma = (1.0 + 0.2 * torch.randn(d, generator=g)).to(dtype)
    layer = vb.Layer(N, T, d, d, dtype, vb.GEMM_FMA)
    Xc, dYc, gc = X.cuda(), dY.cuda(), gamma.cuda()
    kept = torch.zeros(N, dtype=torch.int32, device="cuda"); cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    a_out = torch.empty(N * T, layer.chain_parts(), dtype=torch.float32, device="cuda")
    for seed, rho in ((1, 0.5), (2, 1.0), (2 ** 40 + 3, 0.3)):
        dX, dg, db = layer.layernorm_bwd(Xc, gc, dYc, rho, seed, kept_out=kept, kept_cnt_out=cnt, a_out=a_out)
        s = layer.last_sampling()
        own = o.layernorm_bwd(np64(X), np64(gamma), np64(dY), N, T, f32(rho), seed)
        assert np.allclose(np64(s.g), own["g"], rtol=1e-5) and np.allclose(np64(s.p), own["p32"], rtol=1e-5, atol=1e-12)
        ref = o.layernorm_bwd(np64(X), np64(gamma), np64(dY), N, T, f32(rho), seed, p_override=s.p.cpu().numpy())
        assert np.array_equal(s.idxA.cpu().numpy(), np.flatnonzero(ref["keepA"]))             # masks: bit-exact
        assert np.array_equal(kept[:int(cnt.item())].cpu().numpy(), np.flatnonzero(ref["keepA"]))
        assert rel_fro(np64(dX), ref["dX"]) <= tol
        assert rel_fro(np64(dg), ref["dgamma"]) <= tol and rel_fro(np64(db), ref["dbeta"]) <= tol
        assert not np64(dX)[np.repeat(~ref["keepA"], T)].any()
        assert np.allclose(np64(a_out).sum(axis=1), (np64(dX) ** 2).sum(axis=1), rtol=1e-5, atol=1e-30)
        if rho == 1.0:
            assert ref["keepA"].all()
    # handed down a chain: only the alive data are read, dropped rows may be left unwritten
    alive = torch.tensor([0, 2], dtype=torch.int32, device="cuda")
    acnt = torch.tensor([2], dtype=torch.int32, device="cuda")
    dX = torch.full((N * T, d), 7.0, dtype=dtype, device="cuda")
    layer.layernorm_bwd(Xc, gc, dYc, 0.9, 11, dX=dX, alive_in=alive, alive_cnt_in=acnt, skip_dropped_rows=True)
    s = layer.last_sampling()
    assert set(s.idxA.cpu().tolist()) <= {0, 2} and s.cntA >= 1
    keep = np.zeros(N, bool); keep[s.idxA.cpu().numpy()] = True
    assert torch.all(dX[torch.from_numpy(np.repeat(~keep, T)).cuda()] == 7.0)
    assert layer.device_status() == 0
    layer.close()
