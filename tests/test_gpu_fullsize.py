"""GPU parity at the full sizes of the benchmark workloads, in the launch configuration bench.py
times (automatic kernel choice, library-computed probabilities).

Two comparisons per call, so that no test can pass without comparing the products:
  (1) the library's g, p, w, q against the oracle's own (1e-5 / 2e-5 relative); where a mask bit then
      differs, its uniform must lie within that tolerance of its threshold;
  (2) the oracle is given the library's float32 p and q (its override arguments): masks and index lists
      must then be bit-exact, and dX, dW are compared in full - in Frobenius norm (the stated contract
      and a tighter regression gate), row by row, and dropped rows must be exactly zero.
"""
import numpy as np
import pytest
import torch

from oracle import vcas_oracle as o
from paper_2402_17227_b200 import binding as vb
from paper_2402_17227_b200 import build as vbuild
from paper_2402_17227_b200 import inputs
from tests.util import f32, np64, rel_fro

pytestmark = pytest.mark.gpu
TOL = 2e-2            # the contract: bf16 inputs, fp32 accumulation, relative Frobenius error
GATE_DX = 5e-3        # regression gates, 3x the errors measured: 1.66e-3 (the bf16 rounding of dX) and
GATE_DW = 5e-3        # 1.6-1.7e-3 (the bf16 rounding of the rescaled rows that enter the weight-gradient product)
ROW_TOL = 1e-2        # every single row of dX and of dW, relative 2-norm error


@pytest.fixture(scope="module", autouse=True)
def _lib():
    vbuild.build()
    vb.lib()


def f32np(t):
    return t.float().numpy()


def borderline(diff_idx, u24, prob, tol):
    """Indices whose mask bit differs must have their uniform within `tol` (relative) of the threshold."""
    u = u24[diff_idx].astype(np.float64) / 2 ** 24
    return np.all(np.abs(u - prob[diff_idx]) <= tol * prob[diff_idx] + 2.0 ** -23)


def row_errors(got, ref):
    """Relative 2-norm error of every row (rows whose reference is zero must be zero)."""
    num = np.linalg.norm(got - ref, axis=1)
    den = np.linalg.norm(ref, axis=1)
    zero = den == 0
    assert not got[zero].any()
    return num[~zero] / den[~zero]


def check_call(layer, X, dY, W, rho, nu, seed, dX, dW, H=None):
    """Checks one library call (already made; outputs dX, dW) against the oracle.  Returns the oracle's
    scores / masks computed from the library's probabilities."""
    N, T = layer.N, layer.T
    s = layer.last_sampling()
    Xf, dYf, Wf = f32np(X), f32np(dY), f32np(W)
    # (1) the library's probabilities against the oracle's own
    own = o.scores_and_masks_large(Xf, dYf, N, T, f32(rho), f32(nu), seed)
    assert np.allclose(np64(s.g), own["g"], rtol=1e-5, atol=1e-30)
    assert np.allclose(np64(s.p), own["p32"], rtol=1e-5, atol=1e-12)
    p_gpu, q_gpu = s.p.cpu().numpy(), s.q.cpu().numpy()
    # (2) the oracle on the library's p, q: masks and lists bit-exact
    t2 = o.scores_and_masks_large(Xf, dYf, N, T, f32(rho), f32(nu), seed, p_override=p_gpu, q_override=q_gpu)
    assert np.array_equal(s.idxA.cpu().numpy(), np.flatnonzero(t2["keepA"]))
    assert np.array_equal(s.idxW.cpu().numpy(), np.flatnonzero(t2["keepW"]))
    assert s.cntA == int(t2["keepA"].sum()) and s.cntW == int(t2["keepW"].sum())
    assert np.allclose(np64(s.w), t2["w"], rtol=1e-5, atol=1e-30)
    # ... and where the oracle's own probabilities give another list, the differing bits are borderline
    diffA = np.flatnonzero(own["keepA"] != t2["keepA"])
    assert borderline(diffA, o.uniform24(seed, 0, np.arange(N)), own["p32"].astype(np.float64), 1e-5)
    if len(diffA) == 0:
        assert np.allclose(q_gpu, own["q32"], rtol=2e-5, atol=1e-12)
        diffW = np.flatnonzero(own["keepW"] != t2["keepW"])
        assert borderline(diffW, o.uniform24(seed, 1, np.arange(N * T)), own["q32"].astype(np.float64), 2e-5)
    # products, in full
    dX_ref, dW_ref = o.products_on_kept_rows(Xf, dYf, Wf, p_gpu, q_gpu, t2["keepA"], t2["keepW"], T)
    if H is not None:
        dX_ref = dX_ref * o.gelu_prime(np64(H))
    dX_g, dW_g = np64(dX), np64(dW)
    e_dx, e_dw = rel_fro(dX_g, dX_ref), rel_fro(dW_g, dW_ref)
    assert e_dx <= TOL and e_dw <= TOL
    assert e_dx <= GATE_DX and e_dw <= GATE_DW, (e_dx, e_dw)
    assert not dX_g[np.repeat(~t2["keepA"], T)].any()               # rows of dropped data exactly zero
    if t2["keepA"].any():
        assert row_errors(dX_g, dX_ref).max() <= ROW_TOL
        assert row_errors(dW_g, dW_ref).max() <= ROW_TOL
    return t2


def run_and_check(case, rho, nu, seed):
    X, dY, W = inputs.make_layer(case)
    layer = vb.Layer(case.N, case.T, case.d_in, case.d_out, case.dtype)
    dX, dW = layer.linear_bwd(X.cuda(), dY.cuda(), W.cuda(), rho, nu, seed)
    t2 = check_call(layer, X, dY, W, rho, nu, seed, dX, dW)
    assert 0 < t2["keepA"].sum() <= case.N
    assert layer.device_status() == 0
    layer.close()


def test_bert_base_ffn_up_full_size():
    """BERT-base FFN up-projection, several seeds, and the dense products."""
    case = inputs.CASES["bert_base_ffn_up"]
    for seed in (0, 1, 2):
        run_and_check(case, case.rho, case.nu, seed)
    X, dY, W = inputs.make_layer(case)
    layer = vb.Layer(case.N, case.T, case.d_in, case.d_out, case.dtype)
    dXd, dWd = o.dense_bwd(np64(X), np64(dY), np64(W))
    dX, dW = layer.dense_bwd(X.cuda(), dY.cuda(), W.cuda())
    assert rel_fro(np64(dX), dXd) <= GATE_DX and rel_fro(np64(dW), dWd) <= 1e-4      # no bf16 rounding in dense dW
    assert row_errors(np64(dX), dXd).max() <= ROW_TOL and row_errors(np64(dW), dWd).max() <= 1e-3
    assert layer.device_status() == 0
    layer.close()


def test_vit_mlp_block_two_linears_with_gelu():
    """ViT-base MLP block (N=64, T=197, 768 -> 3072 -> 768): backward through fc2, the GELU Jacobian fused in
    its epilogue, then fc1, whose incoming gradient has zero rows for every datum dropped above (App. E)."""
    fc2 = inputs.CASES["vit_base_mlp_fc2"]
    N, T, hidden, d = fc2.N, fc2.T, fc2.d_in, fc2.d_out
    H = inputs.make_preactivation(fc2, width=hidden)                       # saved pre-activation
    A = torch.nn.functional.gelu(H.float()).to(torch.bfloat16)            # fc2's input
    _, dZ2, W2 = inputs.make_layer(fc2)                                    # dZ2 [R, 768], W2 [768, 3072]
    X1, _, W1 = inputs.make_layer(inputs.CASES["vit_base_mlp_fc1"])        # X1 [R, 768], W1 [3072, 768]
    l2 = vb.Layer(N, T, hidden, d, torch.bfloat16)
    l1 = vb.Layer(N, T, d, hidden, torch.bfloat16)
    rho, nu, seed = fc2.rho, fc2.nu, 11
    dZ1, dW2 = l2.linear_bwd(A.cuda(), dZ2.cuda(), W2.cuda(), rho, nu, seed, H=H.cuda())
    t2 = check_call(l2, A, dZ2, W2, rho, nu, seed, dZ1, dW2, H=H)
    # fc1 consumes the library's own dZ1 (bf16): its dropped data arrive as exact zero rows
    dX1, dW1 = l1.linear_bwd(X1.cuda(), dZ1, W1.cuda(), rho, nu, seed + 1)
    t1 = check_call(l1, X1, dZ1.cpu(), W1, rho, nu, seed + 1, dX1, dW1)
    assert np.all(t1["p32"][~t2["keepA"]] == 0)                            # compounding sparsity
    assert not (t1["keepA"] & ~t2["keepA"]).any() and t1["keepA"].sum() <= t2["keepA"].sum()
    assert l1.device_status() == 0 and l2.device_status() == 0
    l1.close(); l2.close()


@pytest.mark.parametrize("rho,nu,seed", [(0.3, 0.3, 3), (0.5, 0.3, 4)])
def test_llm_mlp_up_full_size(rho, nu, seed):
    """LLM-sized layer (N=8, T=2048, 4096 -> 11008), more tiles than SMs in both products: every row of
    both outputs, including the last tiles of each launch."""
    run_and_check(inputs.CASES["llm_mlp_up"], rho, nu, seed)


@pytest.mark.parametrize("name", ["bert_large_qkv", "bert_large_attn_out", "bert_large_ffn_up", "bert_large_ffn_down"])
@pytest.mark.parametrize("rho,seed", [(0.8, 5), (0.2, 6)])
def test_bert_large_linears_full_size(name, rho, seed):
    """The four linears of a BERT-large block (N=32, T=512) at the keep ratios of a top and of a bottom layer."""
    case = inputs.CASES[name]
    run_and_check(case, rho, case.nu, seed)
