"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs and the same Philox stream."""
import numpy as np
import pytest
import torch

from oracle import vcas_oracle as o
from paper_2402_17227_b200 import binding as vb
from paper_2402_17227_b200 import build as vbuild
from paper_2402_17227_b200 import inputs
from tests.util import f32, np64, rel_fro, tol_for

pytestmark = pytest.mark.gpu

F32, BF16 = torch.float32, torch.bfloat16
PATHS = [("fp32-fma", F32, vb.GEMM_FMA), ("bf16-fma", BF16, vb.GEMM_FMA), ("bf16-tensor", BF16, vb.GEMM_TENSOR)]


@pytest.fixture(scope="module", autouse=True)
def _lib():
    vbuild.build()
    vb.lib()


def small_case(dtype, N, T, d_in, d_out, sigma_A=1.0, sigma_B=0.5, zero_fraction=0.0, seed=1234):
    case = inputs.LayerCase("t", N, T, d_in, d_out, dtype, sigma_A, sigma_B, 0.5, 0.5, data_seed=seed,
                            zero_fraction=zero_fraction)
    return inputs.make_layer(case)


def cuda(*ts):
    return [t.cuda() for t in ts]


# several tiles and a ragged tail in every dimension the kernels tile: T = 197 (128 + 69),
# d_in = 320 (256 + 64), d_out = 192 (3 k-blocks of 64), N = 5
SHAPES = [(5, 197, 320, 192), (6, 64, 128, 256), (3, 130, 64, 64)]


def check_sampling(s, ref, N, T):
    """Scores and probabilities within 1e-5 relative; lists identical unless a mask bit sits within
    that tolerance of its threshold (then the differing index must be such a borderline one)."""
    assert np.allclose(np64(s.g), ref["g"], rtol=1e-5, atol=1e-30)
    assert np.allclose(np64(s.p), ref["p32"], rtol=1e-5, atol=1e-12)
    keepA_gpu = np.zeros(N, bool); keepA_gpu[s.idxA.cpu().numpy()] = True
    diffA = np.flatnonzero(keepA_gpu != ref["keepA"])
    uA = o.uniform24(ref["seed"], 0, np.arange(N)).astype(np.float64) / 2 ** 24
    assert np.all(np.abs(uA[diffA] - ref["p32"][diffA]) <= 1e-5 * ref["p32"][diffA] + 2 ** -24)
    if len(diffA):
        return False
    assert s.cntA == int(ref["keepA"].sum())
    assert np.allclose(np64(s.w), ref["w"], rtol=1e-5, atol=1e-30)
    assert np.allclose(np64(s.q), ref["q32"], rtol=2e-5, atol=1e-12)
    keepW_gpu = np.zeros(N * T, bool); keepW_gpu[s.idxW.cpu().numpy()] = True
    diffW = np.flatnonzero(keepW_gpu != ref["keepW"])
    uW = o.uniform24(ref["seed"], 1, np.arange(N * T)).astype(np.float64) / 2 ** 24
    assert np.all(np.abs(uW[diffW] - ref["q32"][diffW]) <= 2e-5 * ref["q32"][diffW] + 2 ** -24)
    if len(diffW):
        return False
    assert s.cntW == int(ref["keepW"].sum())
    assert np.array_equal(s.idxW.cpu().numpy(), np.flatnonzero(ref["keepW"]))
    return True


@pytest.mark.parametrize("dtype", [F32, BF16])
@pytest.mark.parametrize("shape", SHAPES)
def test_score_matches_oracle(dtype, shape):
    N, T, d_in, d_out = shape
    X, dY, W = small_case(dtype, N, T, d_in, d_out, sigma_A=1.5, sigma_B=1.0)
    layer = vb.Layer(N, T, d_in, d_out, dtype, vb.GEMM_FMA)
    Xc, dYc = cuda(X, dY)
    for seed, rho, nu in [(0, 0.5, 0.5), (7, 0.3, 0.4), (2 ** 40 + 5, 0.8, 0.25)]:
        s = layer.score(Xc, dYc, rho, nu, seed)
        ref = o.linear_bwd(np64(X), np64(dY), np64(W), N, T, f32(rho), f32(nu), seed)
        ref["seed"] = seed
        check_sampling(s, ref, N, T)
        assert np.isclose(float(s.p.sum()), min(N * f32(rho), np.count_nonzero(ref["g"])), rtol=1e-5)
    assert layer.device_status() == 0
    layer.close()


@pytest.mark.parametrize("N,T", [(40, 250), (64, 100), (33, 31), (20, 1000), (1100, 3), (70, 1000)])
def test_score_kernel_variants(N, T):
    """Sizes that select each variant of the sampling kernels: up to 32 data, up to 1024 data, more than 1024 data
    (SampleA in one warp, in one warp with several data per lane, block-wide), and, with 70000 rows at rho = 0.95,
    more SampleW scores than fit one CTA's shared memory (the water-filling then reads them from global memory)."""
    d_in = d_out = 64
    X, dY, W = small_case(BF16, N, T, d_in, d_out, sigma_A=1.5, sigma_B=1.0, zero_fraction=0.1 if N * T < 60000 else 0.0)
    layer = vb.Layer(N, T, d_in, d_out, BF16, vb.GEMM_FMA)
    Xc, dYc = cuda(X, dY)
    for seed, rho, nu in [(1, 0.3, 0.4), (5, 0.6, 0.2)] + ([(2, 0.95, 0.3)] if N * T >= 60000 else []):
        s = layer.score(Xc, dYc, rho, nu, seed)
        ref = o.linear_bwd(np64(X), np64(dY), np64(W), N, T, f32(rho), f32(nu), seed)
        ref["seed"] = seed
        check_sampling(s, ref, N, T)
    assert layer.device_status() == 0
    layer.close()


@pytest.mark.parametrize("n", [1, 31, 1024, 5000, 16384 + 17])
def test_masks_bit_exact_given_oracle_probabilities(n):
    r = np.random.default_rng(n)
    p = r.random(n).astype(np.float32)
    p[r.random(n) < 0.1] = 0.0
    p[r.random(n) < 0.1] = 1.0
    layer = vb.Layer(4, 4, 64, 64, BF16, vb.GEMM_FMA)
    pc = torch.from_numpy(p).cuda()
    for seed, sampler in [(0, 0), (0, 1), (123456789012345, 1), (2 ** 64 - 1, 0)]:
        keep, idx, cnt = layer.mask_from_probs(pc, seed, sampler)
        ref = o.bernoulli_keep(p, seed, sampler)
        assert np.array_equal(keep.cpu().numpy().astype(bool), ref)
        assert np.array_equal(idx.cpu().numpy(), np.flatnonzero(ref))
        assert cnt == int(ref.sum())
    layer.close()


@pytest.mark.parametrize("name,dtype,path", PATHS)
@pytest.mark.parametrize("shape", SHAPES)
def test_linear_bwd_given_oracle_probabilities(name, dtype, path, shape):
    """Fed the oracle's p and q, masks and lists are bit-exact and dX, dW meet the tolerance."""
    N, T, d_in, d_out = shape
    X, dY, W = small_case(dtype, N, T, d_in, d_out, sigma_A=1.5, sigma_B=1.0)
    layer = vb.Layer(N, T, d_in, d_out, dtype, path)
    Xc, dYc, Wc = cuda(X, dY, W)
    for seed, rho, nu in [(3, 0.5, 0.5), (11, 0.3, 0.4)]:
        ref = o.linear_bwd(np64(X), np64(dY), np64(W), N, T, f32(rho), f32(nu), seed)
        p_in = torch.from_numpy(ref["p32"]).cuda()
        q_in = torch.from_numpy(ref["q32"]).cuda()
        dX, dW = layer.linear_bwd(Xc, dYc, Wc, rho, nu, seed, p_in=p_in, q_in=q_in)
        s = layer.last_sampling()
        assert np.array_equal(s.idxA.cpu().numpy(), ref["idxA"])
        assert np.array_equal(s.idxW.cpu().numpy(), ref["idxW"])
        assert rel_fro(np64(dX), ref["dX"]) <= tol_for(dtype), name
        assert rel_fro(np64(dW), ref["dW"]) <= tol_for(dtype), name
        dropped = np.repeat(~ref["keepA"], T)
        assert not np64(dX)[dropped].any()                  # rows of dropped data are exactly zero
    assert layer.device_status() == 0
    layer.close()


@pytest.mark.parametrize("tile_n,split,tile_m", [(256, 3, 1), (128, 2, 1), (64, 5, 1), (256, 16, 1), (256, 1, 1),
                                                 (64, 1, 1), (256, 1, 2), (256, 0, 2), (128, 8, 1), (256, 4, 1)])
def test_tensor_path_split_contraction_and_tile_widths(tile_n, split, tile_m):
    """Every tile width and a contraction cut into slices (combined in a fixed order) give the same
    results within tolerance, for the sampled and the dense products; repeated runs are bit-identical."""
    N, T, d_in, d_out = 5, 197, 320, 448
    X, dY, W = small_case(BF16, N, T, d_in, d_out, sigma_A=1.5, sigma_B=1.0)
    layer = vb.Layer(N, T, d_in, d_out, BF16, vb.GEMM_TENSOR)
    layer.set_tuning(tile_n, tile_n, split, split, tile_m)
    Xc, dYc, Wc = cuda(X, dY, W)
    ref = o.linear_bwd(np64(X), np64(dY), np64(W), N, T, 0.5, 0.5, 4)
    p_in, q_in = torch.from_numpy(ref["p32"]).cuda(), torch.from_numpy(ref["q32"]).cuda()
    dX, dW = layer.linear_bwd(Xc, dYc, Wc, 0.5, 0.5, 4, p_in=p_in, q_in=q_in)
    assert rel_fro(np64(dX), ref["dX"]) <= tol_for(BF16) and rel_fro(np64(dW), ref["dW"]) <= tol_for(BF16)
    assert not np64(dX)[np.repeat(~ref["keepA"], T)].any()
    dX2, dW2 = layer.linear_bwd(Xc, dYc, Wc, 0.5, 0.5, 4, p_in=p_in, q_in=q_in)
    assert torch.equal(dX, dX2) and torch.equal(dW, dW2)
    dXd, dWd = o.dense_bwd(np64(X), np64(dY), np64(W))
    dX3, dW3 = layer.dense_bwd(Xc, dYc, Wc)
    assert rel_fro(np64(dX3), dXd) <= tol_for(BF16) and rel_fro(np64(dW3), dWd) <= tol_for(BF16)
    # the GELU Jacobian under the same tiling (the slice reduction and the unsliced epilogue each apply it), with
    # pre-activations on both sides of the polynomial's clamp at |x| = 5
    H = (2.5 * torch.randn(N * T, d_in, generator=torch.Generator().manual_seed(8))).to(BF16)
    gp = o.gelu_prime(np64(H))
    dX5, dW5 = layer.linear_bwd(Xc, dYc, Wc, 0.5, 0.5, 4, p_in=p_in, q_in=q_in, H=H.cuda())
    assert rel_fro(np64(dX5), ref["dX"] * gp) <= tol_for(BF16) and torch.equal(dW5, dW)
    assert np.abs(np64(dX5) - ref["dX"] * gp).max() <= 2e-2 * np.abs(ref["dX"]).max()
    dX6, _ = layer.dense_bwd(Xc, dYc, Wc, H=H.cuda())
    assert rel_fro(np64(dX6), dXd * gp) <= tol_for(BF16)
    assert layer.device_status() == 0
    layer.close()


@pytest.mark.parametrize("shape,rho,nu", [((48, 512, 512, 512), 0.85, 0.5), ((4, 256, 4096, 2560), 0.75, 0.5)])
def test_tensor_path_whole_waves_and_remainder(shape, rho, nu):
    """Problems of more tiles than SMs with 256-row tiles for whole waves of CTAs and a second launch of sliced
    128-row tiles for the rest (the first shape leaves a remainder in the dX product, the second in the dW
    product): sampled and dense products against the oracle, and bit-identical to a second run."""
    N, T, d_in, d_out = shape
    X, dY, W = small_case(BF16, N, T, d_in, d_out, sigma_A=0.3, sigma_B=0.5)
    layer = vb.Layer(N, T, d_in, d_out, BF16, vb.GEMM_TENSOR)
    layer.set_tuning(256, 256, 0, 0, 3)
    Xc, dYc, Wc = cuda(X, dY, W)
    ref = o.linear_bwd(np64(X), np64(dY), np64(W), N, T, f32(rho), f32(nu), 9)
    p_in, q_in = torch.from_numpy(ref["p32"]).cuda(), torch.from_numpy(ref["q32"]).cuda()
    dX, dW = layer.linear_bwd(Xc, dYc, Wc, rho, nu, 9, p_in=p_in, q_in=q_in)
    s = layer.last_sampling()
    assert np.array_equal(s.idxA.cpu().numpy(), ref["idxA"]) and np.array_equal(s.idxW.cpu().numpy(), ref["idxW"])
    assert rel_fro(np64(dX), ref["dX"]) <= tol_for(BF16) and rel_fro(np64(dW), ref["dW"]) <= tol_for(BF16)
    assert not np64(dX)[np.repeat(~ref["keepA"], T)].any()
    dX2, dW2 = layer.linear_bwd(Xc, dYc, Wc, rho, nu, 9, p_in=p_in, q_in=q_in)
    assert torch.equal(dX, dX2) and torch.equal(dW, dW2)
    dXd, dWd = o.dense_bwd(np64(X), np64(dY), np64(W))
    dX3, dW3 = layer.dense_bwd(Xc, dYc, Wc)
    assert rel_fro(np64(dX3), dXd) <= tol_for(BF16) and rel_fro(np64(dW3), dWd) <= tol_for(BF16)
    # the same through one launch of 128-row tiles: every element within rounding of the other tiling
    layer.set_tuning(256, 256, 1, 1, 1)
    dX4, dW4 = layer.dense_bwd(Xc, dYc, Wc)
    assert rel_fro(np64(dX3), np64(dX4)) <= 1e-2 and rel_fro(np64(dW3), np64(dW4)) <= 1e-4
    assert layer.device_status() == 0
    layer.close()


@pytest.mark.parametrize("N,T", [(160, 16), (128, 24), (40, 8)])
def test_tensor_path_many_data(N, T):
    """Batches of more data than one warp holds in one slot per lane (SampleA's wide variant) and fewer: the
    kept data, the lists and both products against the oracle with given probabilities; with the library's
    own, the dX product's kept data (from the SampleA-only kernel) must be those of the sampling kernel."""
    d_in, d_out = 128, 192
    X, dY, W = small_case(BF16, N, T, d_in, d_out, sigma_A=1.0, sigma_B=0.5)
    layer = vb.Layer(N, T, d_in, d_out, BF16, vb.GEMM_TENSOR)
    Xc, dYc, Wc = cuda(X, dY, W)
    rho, nu, seed = 0.4, 0.5, 21
    ref = o.linear_bwd(np64(X), np64(dY), np64(W), N, T, f32(rho), f32(nu), seed)
    p_in, q_in = torch.from_numpy(ref["p32"]).cuda(), torch.from_numpy(ref["q32"]).cuda()
    dX, dW = layer.linear_bwd(Xc, dYc, Wc, rho, nu, seed, p_in=p_in, q_in=q_in)
    s = layer.last_sampling()
    assert np.array_equal(s.idxA.cpu().numpy(), ref["idxA"]) and np.array_equal(s.idxW.cpu().numpy(), ref["idxW"])
    assert rel_fro(np64(dX), ref["dX"]) <= tol_for(BF16) and rel_fro(np64(dW), ref["dW"]) <= tol_for(BF16)
    kept_rows = np.repeat(ref["keepA"], T)
    assert not np64(dX)[~kept_rows].any()
    # library-computed probabilities: dX's kept data (from its own SampleA) must be the sampler's
    dX2, dW2 = layer.linear_bwd(Xc, dYc, Wc, rho, nu, seed)
    s2 = layer.last_sampling()
    keep2 = np.zeros(N, bool); keep2[s2.idxA.cpu().numpy()] = True
    nz = np64(dX2).reshape(N, -1).any(axis=1)
    assert np.array_equal(nz, keep2 & (np64(dY).reshape(N, -1).any(axis=1)))
    assert layer.device_status() == 0
    layer.close()


@pytest.mark.parametrize("name,dtype,path", PATHS)
def test_linear_bwd_end_to_end(name, dtype, path):
    """No overrides: the library's own probabilities, masks and products against the oracle's."""
    N, T, d_in, d_out = 8, 96, 192, 256
    X, dY, W = small_case(dtype, N, T, d_in, d_out, sigma_A=1.0, sigma_B=0.5)
    layer = vb.Layer(N, T, d_in, d_out, dtype, path)
    Xc, dYc, Wc = cuda(X, dY, W)
    compared = 0
    for seed in range(4):
        dX, dW = layer.linear_bwd(Xc, dYc, Wc, 0.5, 0.5, seed)
        s = layer.last_sampling()
        ref = o.linear_bwd(np64(X), np64(dY), np64(W), N, T, 0.5, 0.5, seed)
        ref["seed"] = seed
        if check_sampling(s, ref, N, T):
            compared += 1
            assert rel_fro(np64(dX), ref["dX"]) <= tol_for(dtype)
            assert rel_fro(np64(dW), ref["dW"]) <= tol_for(dtype)
    assert compared >= 3
    assert layer.device_status() == 0
    layer.close()


@pytest.mark.parametrize("name,dtype,path", PATHS)
def test_ratio_one_is_exact_backprop(name, dtype, path):
    N, T, d_in, d_out = 4, 150, 128, 192
    X, dY, W = small_case(dtype, N, T, d_in, d_out)
    layer = vb.Layer(N, T, d_in, d_out, dtype, path)
    Xc, dYc, Wc = cuda(X, dY, W)
    dX, dW = layer.linear_bwd(Xc, dYc, Wc, 1.0, 1.0, 5)
    s = layer.last_sampling()
    assert s.cntA == N and s.cntW == N * T
    assert torch.all(s.p == 1) and torch.all(s.q == 1)
    dXd, dWd = o.dense_bwd(np64(X), np64(dY), np64(W))
    assert rel_fro(np64(dX), dXd) <= tol_for(dtype) and rel_fro(np64(dW), dWd) <= tol_for(dtype)
    dX2, dW2 = layer.dense_bwd(Xc, dYc, Wc)
    assert rel_fro(np64(dX2), dXd) <= tol_for(dtype) and rel_fro(np64(dW2), dWd) <= tol_for(dtype)
    layer.close()


@pytest.mark.parametrize("name,dtype,path", PATHS)
def test_degenerate_inputs(name, dtype, path):
    N, T, d_in, d_out = 6, 70, 64, 128
    layer = vb.Layer(N, T, d_in, d_out, dtype, path)
    # all-zero gradient: nothing kept, outputs exactly zero, no error
    X, dY, W = small_case(dtype, N, T, d_in, d_out)
    Xc, dYc, Wc = cuda(X, torch.zeros_like(dY), W)
    dX = torch.full((N * T, d_in), 3.0, dtype=dtype, device="cuda")
    dW = torch.full((d_out, d_in), 3.0, dtype=torch.float32, device="cuda")
    layer.linear_bwd(Xc, dYc, Wc, 0.5, 0.5, 1, dX=dX, dW=dW)
    s = layer.last_sampling()
    assert s.cntA == 0 and s.cntW == 0 and not dX.any() and not dW.any()
    # most data already dropped upstream (zero rows): the survivors saturate at p = 1
    X, dY, W = small_case(dtype, N, T, d_in, d_out, zero_fraction=0.7, seed=77)
    Xc, dYc, Wc = cuda(X, dY, W)
    dX, dW = layer.linear_bwd(Xc, dYc, Wc, 0.9, 0.5, 2)
    s = layer.last_sampling()
    ref = o.linear_bwd(np64(X), np64(dY), np64(W), N, T, f32(0.9), 0.5, 2)
    nz = ref["g"] > 0
    assert 0 < nz.sum() < N * 0.9
    assert np.array_equal(np64(s.p), nz.astype(np.float64))
    assert np.array_equal(s.idxA.cpu().numpy(), np.flatnonzero(nz))
    ref["seed"] = 2
    if check_sampling(s, ref, N, T):
        assert rel_fro(np64(dX), ref["dX"]) <= tol_for(dtype) and rel_fro(np64(dW), ref["dW"]) <= tol_for(dtype)
    # invalid ratios are rejected on the host
    with pytest.raises(vb.VcasError):
        layer.linear_bwd(Xc, dYc, Wc, 0.0, 0.5, 1)
    with pytest.raises(vb.VcasError):
        layer.linear_bwd(Xc, dYc, Wc, 0.5, 1.5, 1)
    assert layer.device_status() == 0
    layer.close()


@pytest.mark.parametrize("name,dtype,path", PATHS)
def test_gelu_jacobian_epilogue(name, dtype, path):
    N, T, d_in, d_out = 4, 100, 128, 64
    X, dY, W = small_case(dtype, N, T, d_in, d_out)
    H = torch.randn(N * T, d_in, generator=torch.Generator().manual_seed(3)).to(dtype)
    layer = vb.Layer(N, T, d_in, d_out, dtype, path)
    Xc, dYc, Wc, Hc = cuda(X, dY, W, H)
    ref = o.linear_bwd(np64(X), np64(dY), np64(W), N, T, 0.5, 0.5, 9)
    dX, dW = layer.linear_bwd(Xc, dYc, Wc, 0.5, 0.5, 9, p_in=torch.from_numpy(ref["p32"]).cuda(),
                              q_in=torch.from_numpy(ref["q32"]).cuda(), H=Hc)
    assert rel_fro(np64(dX), ref["dX"] * o.gelu_prime(np64(H))) <= tol_for(dtype)
    assert rel_fro(np64(dW), ref["dW"]) <= tol_for(dtype)
    # the exact backward with the same Jacobian factor (vcas_dense_bwd_ex)
    dXd, dWd = o.dense_bwd(np64(X), np64(dY), np64(W))
    dX2, dW2 = layer.dense_bwd(Xc, dYc, Wc, H=Hc)
    assert rel_fro(np64(dX2), dXd * o.gelu_prime(np64(H))) <= tol_for(dtype)
    assert rel_fro(np64(dW2), dWd) <= tol_for(dtype)
    layer.close()


def test_gelu_jacobian_values_on_the_tensor_path():
    """The tensor path evaluates GELU' as a polynomial.  With dY = 1 and W = 1/d_out the product is exactly 1, so
    the dense backward with H returns GELU'(H) rounded to bf16: every value, over -9 <= x <= 9 in steps of 2^-6,
    must lie within the bf16 rounding (half a unit in the last of 8 significant bits: 2^-8 relative) plus 1e-4 of the erf form."""
    N, T, d_in, d_out = 2, 128, 256, 64
    xs = torch.arange(-9.0, 9.0, 2.0 ** -6)
    H = xs.repeat((N * T * d_in + xs.numel() - 1) // xs.numel())[:N * T * d_in].reshape(N * T, d_in).to(BF16)
    dY = torch.ones(N * T, d_out, dtype=BF16)
    W = torch.full((d_out, d_in), 1.0 / d_out, dtype=BF16)
    X = torch.zeros(N * T, d_in, dtype=BF16)
    layer = vb.Layer(N, T, d_in, d_out, BF16, vb.GEMM_TENSOR)
    for tune in ((0, 0, 0, 0, 0), (256, 256, 1, 1, 2), (128, 128, 1, 1, 1)):
        layer.set_tuning(*tune)
        dX, _ = layer.dense_bwd(X.cuda(), dY.cuda(), W.cuda(), H=H.cuda())
        ref = o.gelu_prime(np64(H))
        err = np.abs(np64(dX) - ref)
        assert np.all(err <= 2.0 ** -8 * np.abs(ref) + 1e-4), float(err.max())
    assert layer.device_status() == 0
    layer.close()


@pytest.mark.parametrize("name,dtype,path", PATHS)
def test_variance_probe_matches_oracle(name, dtype, path):
    N, T, d_in, d_out, M = 8, 40, 64, 128, 3
    case = inputs.LayerCase("p", N, T, d_in, d_out, dtype, 1.0, 0.5, 0.5, 0.5)
    batches = [inputs.make_layer(case, batch=i) for i in range(M)]
    W = batches[0][2]
    cfg = vb.default_config()
    cfg.alpha = 0.05
    layer = vb.Layer(N, T, d_in, d_out, dtype, path, cfg)
    Xs = [b[0].cuda() for b in batches]
    dYs = [b[1].cuda() for b in batches]
    out = layer.variance_probe(Xs, dYs, W.cuda(), 0.5, 0.5, 0.75, 42).cpu().numpy()
    ref = o.variance_probe([np64(b[0]) for b in batches], [np64(b[1]) for b in batches], np64(W), N, T, 0.5, 0.5,
                           s=0.75, alpha=f32(0.05), seed=42)
    tol = 1e-4 if dtype == F32 else 2e-2
    assert out[0] == pytest.approx(ref["V_s"], rel=tol)
    assert out[1] == pytest.approx(ref["V_act"], rel=tol)
    assert out[2] == pytest.approx(ref["V_w"], rel=1e-4)
    assert out[3] == pytest.approx(ref["p_lo"], abs=1e-6) and out[4] == pytest.approx(ref["p_hi"], abs=1e-6)
    assert layer.device_status() == 0
    with pytest.raises(vb.VcasError):
        layer.variance_probe(Xs[:1], dYs[:1], W.cuda(), 0.5, 0.5, 0.75, 42)       # M >= 2
    layer.close()


def test_unbiasedness_on_gpu():
    """Mean over seeds of the sampled gradients approaches the exact ones at the 1/sqrt(n) rate."""
    N, T, d_in, d_out = 8, 16, 64, 64
    X, dY, W = small_case(F32, N, T, d_in, d_out)
    layer = vb.Layer(N, T, d_in, d_out, F32, vb.GEMM_FMA)
    Xc, dYc, Wc = cuda(X, dY, W)
    dXd, dWd = layer.dense_bwd(Xc, dYc, Wc)
    dXd, dWd = dXd.double(), dWd.double()
    accX = torch.zeros_like(dXd); accW = torch.zeros_like(dWd)
    dX = torch.empty(N * T, d_in, device="cuda"); dW = torch.empty(d_out, d_in, device="cuda")
    err = {}
    for s in range(2000):
        layer.linear_bwd(Xc, dYc, Wc, 0.5, 0.5, s, dX=dX, dW=dW)
        accX += dX; accW += dW
        if s + 1 in (20, 2000):
            err[s + 1] = (float(((accX / (s + 1) - dXd) ** 2).sum()), float(((accW / (s + 1) - dWd) ** 2).sum()))
    for k in range(2):
        slope = np.log(err[2000][k] / err[20][k]) / np.log(100.0)
        assert -1.6 < slope < -0.4, (k, err)
    layer.close()


def test_interleaved_calls_on_two_handles_repeat_bitwise():
    """Sampled, dense and probe calls of two layers, interleaved on two streams for many rounds: every round
    reproduces the first bit for bit (the kernels keep counters in the workspace between launches - slice
    tickets, work counters, probe accumulators - which each launch must leave re-armed), and no wait times out."""
    shapes = [(48, 512, 512, 256), (40, 64, 256, 640)]      # the first has more tiles than SMs (work counter)
    layers, data, first = [], [], []
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for (N, T, d_in, d_out) in shapes:
        X, dY, W = small_case(BF16, N, T, d_in, d_out, sigma_A=1.0, sigma_B=0.5)
        layers.append(vb.Layer(N, T, d_in, d_out, BF16, vb.GEMM_TENSOR))
        data.append(cuda(X, dY, W))
    layers[0].set_tuning(256, 256, 0, 0, 3)        # whole waves + remainder on the first, automatic on the second
    torch.cuda.synchronize()
    for rnd in range(12):
        outs = []
        for k, (layer, (X, dY, W)) in enumerate(zip(layers, data)):
            with torch.cuda.stream(streams[k]):
                dX, dW = layer.linear_bwd(X, dY, W, 0.5, 0.5, 17 + k)
                dXd, dWd = layer.dense_bwd(X, dY, W)
                pr = layer.variance_probe([X, X], [dY, dY], W, 0.5, 0.5, 0.5, 99)
                outs.append((dX.clone(), dW.clone(), dXd.clone(), dWd.clone(), pr.clone()))
        torch.cuda.synchronize()
        if rnd == 0:
            first = outs
        else:
            for a, b in zip(first, outs):
                for x, y in zip(a, b):
                    assert torch.equal(x, y)
    for layer in layers:
        assert layer.device_status() == 0
        layer.close()
