"""vcas_score_static, the entry point for callers that cannot allocate device memory (code
inside a memory-pool region, a real-time loop, a plug-in with a fixed budget): it must give
what vcas_score gives, on consecutive calls that reuse its fixed scratch array, refuse sizes
beyond that array, and leave the amount of free device memory unchanged.  Collected last on
purpose (file name), and self-contained so that it also passes alone in a fresh process."""
import numpy as np
import pytest
import torch

from oracle import vcas_oracle as o
from paper_2402_17227_b200 import binding as vb
from paper_2402_17227_b200 import build as vbuild
from paper_2402_17227_b200 import inputs
from tests.util import f32, np64

pytestmark = pytest.mark.gpu


def same(a: vb.Sampling, b: vb.Sampling):
    assert a.cntA == b.cntA and a.cntW == b.cntW
    assert torch.equal(a.idxA, b.idxA) and torch.equal(a.idxW, b.idxW)          # index work: bit-exact
    for x, y, tol in ((a.g, b.g, 1e-5), (a.p, b.p, 1e-5), (a.w, b.w, 1e-5), (a.q, b.q, 2e-5)):
        assert np.allclose(np64(x), np64(y), rtol=tol, atol=1e-30)


def against_oracle(got: vb.Sampling, X, dY, N, T, rho, nu, seed):
    """The static entry point against the CPU oracle directly: scores within tolerance, and the lists
    bit-exact for the oracle fed the returned float32 probabilities."""
    own = o.scores_and_masks_large(X.float().cpu().numpy(), dY.float().cpu().numpy(), N, T, f32(rho), f32(nu), seed)
    assert np.allclose(np64(got.g), own["g"], rtol=1e-5, atol=1e-30)
    assert np.allclose(np64(got.p), own["p32"], rtol=1e-5, atol=1e-12)
    t2 = o.scores_and_masks_large(X.float().cpu().numpy(), dY.float().cpu().numpy(), N, T, f32(rho), f32(nu), seed,
                                  p_override=got.p.cpu().numpy(), q_override=got.q.cpu().numpy())
    assert np.array_equal(got.idxA.cpu().numpy(), np.flatnonzero(t2["keepA"]))
    assert np.array_equal(got.idxW.cpu().numpy(), np.flatnonzero(t2["keepW"]))
    assert np.allclose(np64(got.w), t2["w"], rtol=1e-5, atol=1e-30)


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
    against_oracle(got1, X1, dY1, N, T, 0.3, 0.4, 5)
    assert 0 < got1.cntA < N and 0 < got1.cntW < N * T
    N2, T2 = 5, 77
    X2, dY2, _ = [t.cuda() for t in inputs.make_layer(case, batch=1, N=N2, T=T2)]
    layer2 = vb.Layer(N2, T2, d_in, d_out, dtype, vb.GEMM_FMA)
    got2 = vb.score_static(X2, dY2, N2, T2, 0.5, 0.25, seed=2 ** 40 + 9)
    same(got2, layer2.score(X2, dY2, 0.5, 0.25, seed=2 ** 40 + 9))
    against_oracle(got2, X2, dY2, N2, T2, 0.5, 0.25, 2 ** 40 + 9)
    # and the first problem again: nothing of the second call leaks into it
    same(vb.score_static(X1, dY1, N, T, 0.3, 0.4, seed=5), got1)
    layer.close(); layer2.close()


def test_static_score_with_many_data():
    """More data than the single-warp SampleA serves (N > 1024): the general sampling path on the fixed array."""
    vbuild.build()
    N, T, d_in, d_out = 1500, 4, 64, 64
    case = inputs.LayerCase("nb", N, T, d_in, d_out, torch.bfloat16, 1.0, 0.5, 0.4, 0.5)
    X, dY, _ = [t.cuda() for t in inputs.make_layer(case)]
    layer = vb.Layer(N, T, d_in, d_out, torch.bfloat16, vb.GEMM_FMA)
    for _ in range(2):
        got = vb.score_static(X, dY, N, T, 0.4, 0.5, seed=77)
        same(got, layer.score(X, dY, 0.4, 0.5, seed=77))
    against_oracle(got, X, dY, N, T, 0.4, 0.5, 77)
    layer.close()


def test_static_score_allocates_no_device_memory():
    """Free device memory (cudaMemGetInfo) is the same before and after calls whose outputs already exist:
    the entry point must not allocate, not even on its first call on the device."""
    vbuild.build()
    N, T, d_in, d_out = 16, 64, 128, 128
    case = inputs.LayerCase("nc", N, T, d_in, d_out, torch.bfloat16, 1.0, 0.5, 0.5, 0.5)
    X, dY, _ = [t.cuda() for t in inputs.make_layer(case)]
    R = N * T
    f = dict(dtype=torch.float32, device="cuda"); i = dict(dtype=torch.int32, device="cuda")
    outs = (torch.empty(N, **f), torch.empty(N, **f), torch.empty(R, **f), torch.empty(R, **f),
            torch.empty(N, **i), torch.zeros(1, **i), torch.empty(R, **i), torch.zeros(1, **i))
    C = vb.C
    ptr = lambda t: C.c_void_p(t.data_ptr())
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for k in range(3):
        rc = vb.lib().vcas_score_static(N, T, d_in, d_out, vb.DTYPE_BF16, ptr(X), ptr(dY), C.c_float(0.5),
                                        C.c_float(0.5), C.c_uint64(k), *[ptr(t) for t in outs],
                                        C.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert rc == 0
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert 0 < int(outs[5].item()) <= N


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
