"""vcas_score_static, the entry point for callers that cannot allocate device memory (code
inside a memory-pool region, a real-time loop, a plug-in with a fixed budget): it must give
what vcas_score gives, on consecutive calls that reuse its fixed scratch array, and refuse
sizes beyond that array.  Collected last on purpose (file name), and self-contained so that it
also passes alone in a fresh process."""
import numpy as np
import pytest
import torch

from paper_2402_17227_b200 import binding as vb
from paper_2402_17227_b200 import build as vbuild
from paper_2402_17227_b200 import inputs
from tests.util import np64

pytestmark = pytest.mark.gpu


def same(a: vb.Sampling, b: vb.Sampling):
    assert a.cntA == b.cntA and a.cntW == b.cntW
    assert torch.equal(a.idxA, b.idxA) and torch.equal(a.idxW, b.idxW)          # index work: bit-exact
    for x, y, tol in ((a.g, b.g, 1e-5), (a.p, b.p, 1e-5), (a.w, b.w, 1e-5), (a.q, b.q, 2e-5)):
        assert np.allclose(np64(x), np64(y), rtol=tol, atol=1e-30)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_score_matches_score_on_two_calls_in_a_row(dtype):
    vbuild.build()
    N, T, d_in, d_out = 12, 150, 192, 320
    case = inputs.LayerCase("na", N, T, d_in, d_out, dtype, 1.5, 1.0, 0.3, 0.4)
    layer = vb.Layer(N, T, d_in, d_out, dtype, vb.GEMM_FMA)
    # first call: a larger problem than the second, so the second finds stale data beyond its own sizes
    X1, dY1, _ = [t.cuda() for t in inputs.make_layer(case, batch=0)]
    got1 = vb.score_static(X1, dY1, N, T, 0.3, 0.4, seed=5)
    same(got1, layer.score(X1, dY1, 0.3, 0.4, seed=5))
    assert 0 < got1.cntA < N and 0 < got1.cntW < N * T
    N2, T2 = 5, 77
    X2, dY2, _ = [t.cuda() for t in inputs.make_layer(case, batch=1, N=N2, T=T2)]
    layer2 = vb.Layer(N2, T2, d_in, d_out, dtype, vb.GEMM_FMA)
    got2 = vb.score_static(X2, dY2, N2, T2, 0.5, 0.25, seed=2 ** 40 + 9)
    same(got2, layer2.score(X2, dY2, 0.5, 0.25, seed=2 ** 40 + 9))
    # and the first problem again: nothing of the second call leaks into it
    same(vb.score_static(X1, dY1, N, T, 0.3, 0.4, seed=5), got1)
    layer.close(); layer2.close()


def test_static_score_rejects_sizes_beyond_its_scratch():
    vbuild.build()
    X = torch.zeros(8, 64, dtype=torch.bfloat16, device="cuda")
    for N, T in ((4097, 1), (129, 128), (1, 16385)):
        with pytest.raises(vb.VcasError) as e:
            ptr = vb.C.c_void_p(X.data_ptr())
            rc = vb.lib().vcas_score_static(N, T, 64, 64, vb.DTYPE_BF16, ptr, ptr,
                                            vb.C.c_float(0.5), vb.C.c_float(0.5), vb.C.c_uint64(0),
                                            None, None, None, None, None, None, None, None, None)
            vb._check(rc, "vcas_score_static")
        assert e.value.code == -2
