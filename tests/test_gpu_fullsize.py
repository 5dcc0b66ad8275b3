"""GPU parity at the full sizes of the benchmark workloads, in the launch configuration bench.py
times (automatic kernel choice, library-computed probabilities)."""
import numpy as np
import pytest
import torch

from oracle import vcas_oracle as o
from paper_2402_17227_b200 import binding as vb
from paper_2402_17227_b200 import build as vbuild
from paper_2402_17227_b200 import inputs
from tests.util import f32, np64, rel_fro

pytestmark = pytest.mark.gpu
TOL = 2e-2          # bf16 inputs, fp32 accumulation


@pytest.fixture(scope="module", autouse=True)
def _lib():
    vbuild.build()
    vb.lib()


def lists_agree(s, keepA, keepW):
    a = np.zeros(keepA.shape[0], bool); a[s.idxA.cpu().numpy()] = True
    w = np.zeros(keepW.shape[0], bool); w[s.idxW.cpu().numpy()] = True
    return np.array_equal(a, keepA) and np.array_equal(w, keepW)


def test_bert_base_ffn_up_full_size():
    """The benchmark's workload, whole outputs against the oracle, several seeds."""
    case = inputs.CASES["bert_base_ffn_up"]
    N, T = case.N, case.T
    X, dY, W = inputs.make_layer(case)
    layer = vb.Layer(N, T, case.d_in, case.d_out, case.dtype)
    Xc, dYc, Wc = X.cuda(), dY.cuda(), W.cuda()
    X64, dY64, W64 = np64(X), np64(dY), np64(W)
    compared = 0
    for seed in (0, 1, 2):
        dX, dW = layer.linear_bwd(Xc, dYc, Wc, case.rho, case.nu, seed)
        s = layer.last_sampling()
        ref = o.linear_bwd(X64, dY64, W64, N, T, f32(case.rho), f32(case.nu), seed)
        assert np.allclose(np64(s.p), ref["p32"], rtol=1e-5, atol=1e-12)
        assert np.allclose(np64(s.q), ref["q32"], rtol=2e-5, atol=1e-12)
        if not lists_agree(s, ref["keepA"], ref["keepW"]):
            continue                       # a mask bit on its threshold (checked in the small-shape tests)
        compared += 1
        assert rel_fro(np64(dX), ref["dX"]) <= TOL and rel_fro(np64(dW), ref["dW"]) <= TOL
        assert not np64(dX)[np.repeat(~ref["keepA"], T)].any()
    assert compared >= 2
    dXd, dWd = o.dense_bwd(X64, dY64, W64)
    dX, dW = layer.dense_bwd(Xc, dYc, Wc)
    assert rel_fro(np64(dX), dXd) <= TOL and rel_fro(np64(dW), dWd) <= TOL
    assert layer.device_status() == 0
    layer.close()


def test_vit_mlp_block_two_linears_with_gelu():
    """ViT-base MLP block (N=64, T=197, 768 -> 3072 -> 768): backward through fc2, the GELU Jacobian fused in
    its epilogue, then fc1, whose incoming gradient has zero rows for every datum dropped above (App. E)."""
    fc2 = inputs.CASES["vit_base_mlp_fc2"]
    N, T, hidden, d = fc2.N, fc2.T, fc2.d_in, fc2.d_out
    R = N * T
    H = inputs.make_preactivation(fc2, width=hidden)                       # saved pre-activation
    A = torch.nn.functional.gelu(H.float()).to(torch.bfloat16)            # fc2's input
    _, dZ2, W2 = inputs.make_layer(fc2)                                    # dZ2 [R, 768], W2 [768, 3072]
    X1, _, W1 = inputs.make_layer(inputs.CASES["vit_base_mlp_fc1"])        # X1 [R, 768], W1 [3072, 768]
    l2 = vb.Layer(N, T, hidden, d, torch.bfloat16)
    l1 = vb.Layer(N, T, d, hidden, torch.bfloat16)
    rho, nu, seed = fc2.rho, fc2.nu, 11
    dZ1, dW2 = l2.linear_bwd(A.cuda(), dZ2.cuda(), W2.cuda(), rho, nu, seed, H=H.cuda())
    s2 = l2.last_sampling()
    ref2 = o.linear_bwd(np64(A), np64(dZ2), np64(W2), N, T, f32(rho), f32(nu), seed)
    assert lists_agree(s2, ref2["keepA"], ref2["keepW"])
    dZ1_ref = ref2["dX"] * o.gelu_prime(np64(H))
    assert rel_fro(np64(dZ1), dZ1_ref) <= TOL and rel_fro(np64(dW2), ref2["dW"]) <= TOL
    # fc1 consumes the library's own dZ1 (bf16): its dropped data arrive as exact zero rows
    dX1, dW1 = l1.linear_bwd(X1.cuda(), dZ1, W1.cuda(), rho, nu, seed + 1)
    s1 = l1.last_sampling()
    ref1 = o.linear_bwd(np64(X1), np64(dZ1), np64(W1), N, T, f32(rho), f32(nu), seed + 1)
    assert np.all(ref1["p32"][~ref2["keepA"]] == 0)                       # compounding sparsity
    assert s1.cntA <= s2.cntA
    assert lists_agree(s1, ref1["keepA"], ref1["keepW"])
    assert rel_fro(np64(dX1), ref1["dX"]) <= TOL and rel_fro(np64(dW1), ref1["dW"]) <= TOL
    assert l1.device_status() == 0 and l2.device_status() == 0
    l1.close(); l2.close()


def check_sampled_outputs(case, rho, nu, seed):
    """Probabilities and lists in full, dX and dW on sampled rows that the oracle computes one by one."""
    N, T, d_in, d_out = case.N, case.T, case.d_in, case.d_out
    X, dY, W = inputs.make_layer(case)
    layer = vb.Layer(N, T, d_in, d_out, case.dtype)
    dX, dW = layer.linear_bwd(X.cuda(), dY.cuda(), W.cuda(), rho, nu, seed)
    s = layer.last_sampling()
    Xf, dYf, Wf = X.float().numpy(), dY.float().numpy(), W.float().numpy()
    a, b = o.row_sqnorms_chunked(dYf), o.row_sqnorms_chunked(Xf)
    g = o.datum_norms(a, N, T)
    p32 = o.capped_prop(g, N * f32(rho)).astype(np.float32)
    keepA = o.bernoulli_keep(p32, seed, 0)
    lev = np.where(np.repeat(keepA, T), np.sqrt(a) / np.repeat(np.maximum(p32, 1e-30), T).astype(np.float64), 0.0) * np.sqrt(b)
    q32 = o.capped_prop(lev, f32(nu) * T * int(keepA.sum())).astype(np.float32)
    keepW = o.bernoulli_keep(q32, seed, 1)
    assert np.allclose(np64(s.g), g, rtol=1e-5)
    assert np.allclose(np64(s.p), p32, rtol=1e-5, atol=1e-12)
    assert np.allclose(np64(s.q), q32, rtol=2e-5, atol=1e-12)
    assert 0 < keepA.sum() <= N
    if not lists_agree(s, keepA, keepW):
        layer.close()
        return False                       # a mask bit on its threshold (checked in the small-shape tests)
    r = np.random.default_rng(0)
    kept_rows = np.flatnonzero(np.repeat(keepA, T))
    rows = list(r.choice(kept_rows, 6, replace=False))
    if (~keepA).any():
        rows += list(r.choice(np.flatnonzero(np.repeat(~keepA, T)), 2))
    ref_rows = o.dX_rows(dYf, Wf, p32, keepA, T, rows)
    assert rel_fro(np64(dX[torch.tensor(rows, device="cuda")]), ref_rows) <= TOL
    outs = list(r.choice(d_out, 6, replace=False)) + [0, d_out - 1]
    ref_outs = o.dW_rows(dYf, Xf, p32, q32, keepW, T, outs)
    assert rel_fro(np64(dW[torch.tensor(outs, device="cuda")]), ref_outs) <= TOL
    # dropped data: whole rows exactly zero; the kept count matches
    assert not dX.view(N, T, d_in)[torch.from_numpy(~keepA).cuda()].any()
    assert s.cntW == int(keepW.sum())
    assert layer.device_status() == 0
    layer.close()
    return True


def test_llm_mlp_up_full_size_sampled_outputs():
    """LLM-sized layer (N=8, T=2048, 4096 -> 11008), more tiles than SMs in both products."""
    assert check_sampled_outputs(inputs.CASES["llm_mlp_up"], 0.5, 0.3, 3)


@pytest.mark.parametrize("name", ["bert_large_qkv", "bert_large_attn_out", "bert_large_ffn_up", "bert_large_ffn_down"])
def test_bert_large_linears_full_size_sampled_outputs(name):
    """The four linears of a BERT-large block (N=32, T=512) at the keep ratios of a top and of a bottom layer."""
    case = inputs.CASES[name]
    agreed = 0
    for rho, seed in ((0.8, 5), (0.2, 6)):
        agreed += check_sampled_outputs(case, rho, case.nu, seed)
    assert agreed >= 1
