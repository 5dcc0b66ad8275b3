"""A stack of linear layers run with the chain entry point (vcas_linear_bwd_chain): every call is checked
against the oracle on the tensors that call consumed, so the scores a layer receives from the layer above
(row square-norms from the dX epilogue, the list of data still alive) must be exactly what re-reading its
incoming gradient would give.  Then Alg. 1 over the stack: probe, ratio update, next pass."""
import numpy as np
import pytest
import torch

from oracle import vcas_oracle as o
from paper_2402_17227_b200 import binding as vb
from paper_2402_17227_b200 import build as vbuild
from paper_2402_17227_b200 import inputs
from paper_2402_17227_b200.stack import LinearStack, StackLayer
from tests.util import f32, np64, rel_fro

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


def make_block_layers(N, T, d, ffn, qkv, block, variants, dev, dtype=BF16):
    """The four linears of one transformer block in backward order: FFN down (with the GELU in front of it), FFN
    up (chained to it), attention output, QKV.  Every linear draws its own synthetic tensors."""
    def case(name, d_in, d_out, k):
        return inputs.LayerCase(name, N, T, d_in, d_out, dtype, 1.0, 0.5, 0.5, 0.5, data_seed=5000 + 10 * block + k)
    out = []
    specs = [("ffn_down", ffn, d, True, False), ("ffn_up", d, ffn, False, True), ("attn_out", d, d, False, False),
             ("qkv", d, qkv, False, False)]
    for k, (name, d_in, d_out, gelu, chained) in enumerate(specs):
        c = case(name, d_in, d_out, k)
        batches = [inputs.make_layer(c, batch=b) for b in range(variants)]
        H = None
        Xs = [b[0].to(dev) for b in batches]
        if gelu:
            Hs = [inputs.make_preactivation(c, batch=b, width=d_in) for b in range(variants)]
            H = [h.to(dev) for h in Hs]
            Xs = [torch.nn.functional.gelu(h.float()).to(dtype).to(dev) for h in Hs]
        out.append(StackLayer(f"b{block}.{name}", d_in, d_out, batches[0][2].to(dev), Xs,
                              [b[1].to(dev) for b in batches], H=H, chained=chained))
    return out


def check_layer(L, X, dY, alive_prev, rho, nu, seed, T, N):
    """One chain call against the oracle on the same tensors.  alive_prev: bool [N] data the layer above kept."""
    h = L.handle
    s = h.last_sampling()
    dYz = dY.float().cpu().numpy().copy()
    if alive_prev is not None:                      # data dropped above are zero by definition, whatever dY holds
        dYz[np.repeat(~alive_prev, T)] = 0.0
    Xf, Wf = X.float().cpu().numpy(), L.W.float().cpu().numpy()
    own = o.scores_and_masks_large(Xf, dYz, N, T, f32(rho), f32(nu), seed)
    assert np.allclose(np64(s.g), own["g"], rtol=1e-5, atol=1e-30)
    assert np.allclose(np64(s.p), own["p32"], rtol=1e-5, atol=1e-12)
    if alive_prev is not None:
        assert not np64(s.p)[~alive_prev].any()
    p_gpu, q_gpu = s.p.cpu().numpy(), s.q.cpu().numpy()
    t2 = o.scores_and_masks_large(Xf, dYz, N, T, f32(rho), f32(nu), seed, p_override=p_gpu, q_override=q_gpu)
    assert np.array_equal(s.idxA.cpu().numpy(), np.flatnonzero(t2["keepA"]))
    assert np.array_equal(s.idxW.cpu().numpy(), np.flatnonzero(t2["keepW"]))
    cnt = int(L.kept_cnt.item())
    assert np.array_equal(L.kept[:cnt].cpu().numpy(), np.flatnonzero(t2["keepA"]))
    dX_ref, dW_ref = o.products_on_kept_rows(Xf, dYz, Wf, p_gpu, q_gpu, t2["keepA"], t2["keepW"], T)
    if L.H is not None:
        dX_ref = dX_ref * o.gelu_prime(np64(L.H[0]))
    assert rel_fro(np64(L.dX), dX_ref) <= 5e-3 and rel_fro(np64(L.dW), dW_ref) <= 5e-3
    assert not np64(L.dX)[np.repeat(~t2["keepA"], T)].any()
    if L.a_out is not None:                         # the epilogue's row square-norms of the stored dX
        a = np64(L.a_out).sum(axis=1)
        assert np.allclose(a, (np64(L.dX) ** 2).sum(axis=1), rtol=1e-5, atol=1e-30)
    return t2["keepA"]


@pytest.mark.parametrize("T", [64, 197])
def test_stack_with_chained_scores_matches_oracle(T):
    vbuild.build()
    dev = torch.device("cuda")
    N, d, ffn, qkv = 8, 256, 512, 384
    layers = []
    for block in (1, 0):                            # backward order: the upper block first
        layers += make_block_layers(N, T, d, ffn, qkv, block, 1, dev)
    stack = LinearStack(layers, N, T, gemm_path=vb.GEMM_TENSOR)
    L = len(layers)
    rho = np.linspace(0.8, 0.3, L)
    nu = np.full(L, 0.5)
    for step in range(2):
        # run the pass layer by layer so that every call can be checked on the tensors it consumed
        alive = None
        prev = None
        for i, lay in enumerate(layers):
            kw = {}
            if prev is not None:
                kw.update(alive_in=prev.kept, alive_cnt_in=prev.kept_cnt)
            dY = prev.dX.clone() if lay.chained else lay.dY[0]
            if lay.chained:
                kw.update(a_in=prev.a_out, a_in_parts=prev.handle.chain_parts())
            seed = step * L + i
            lay.handle.linear_bwd_chain(lay.X[0], dY, lay.W, float(rho[i]), float(nu[i]), seed, lay.dX, lay.dW,
                                        H=lay.H[0] if lay.H is not None else None, a_out=lay.a_out,
                                        kept_out=lay.kept, kept_cnt_out=lay.kept_cnt, **kw)
            alive = check_layer(lay, lay.X[0], dY, alive, rho[i], nu[i], seed, T, N)
            prev = lay
        assert 0 < alive.sum() < N                  # the gradient got sparser down the stack
        # the same pass through LinearStack.backward gives the same bits
        keep = [(l.dW.clone(), l.kept.clone(), l.kept_cnt.clone()) for l in layers]
        stack.backward(rho, nu, seed=step)
        for l, (dW, kept, cnt) in zip(layers, keep):
            assert torch.equal(l.dW, dW) and torch.equal(l.kept_cnt, cnt)
            assert torch.equal(l.kept[:int(cnt.item())], kept[:int(cnt.item())])
    assert stack.device_status() == 0
    stack.close()


def test_stack_adaptation_follows_the_oracle():
    """Alg. 1 over a two-block stack: the library's probe + update trajectory of (s, rho_l, nu_l) against the
    oracle's, with sampled passes in between."""
    vbuild.build()
    dev = torch.device("cuda")
    N, T, d, ffn, qkv, M = 8, 32, 128, 256, 192, 2
    cfg = vb.default_config()
    cfg.M = M
    cfg.alpha, cfg.beta, cfg.tau_act, cfg.tau_w = 0.05, 0.8, 0.5, 0.5
    layers = []
    for block in (1, 0):
        layers += make_block_layers(N, T, d, ffn, qkv, block, M, dev)
    stack = LinearStack(layers, N, T, config=cfg, gemm_path=vb.GEMM_TENSOR)
    L = len(layers)
    # state in Alg. 1's layer order (index 0 = lowest layer); the stack runs top layer first
    s_g, rho_g, nu_g = 1.0, [1.0] * L, [1.0] * L
    s_o, rho_o, nu_o = 1.0, np.ones(L), np.ones(L)
    kw = dict(tau_act=f32(0.5), tau_w=f32(0.5), alpha=f32(0.05), beta=f32(0.8))
    moved = False
    for period in range(4):
        V = stack.probe(rho_g[::-1], nu_g[::-1], s_g, seed=100 * period).cpu().numpy()[::-1]     # -> layer order
        Vo = np.zeros((L, 5))
        for i, lay in enumerate(layers):
            l = L - 1 - i
            ref = o.variance_probe([np64(x) for x in lay.X], [np64(y) for y in lay.dY], np64(lay.W), N, T,
                                   f32(rho_o[l]), f32(nu_o[l]), s=f32(s_o), alpha=f32(0.05), seed=100 * period + i)
            Vo[l] = [ref["V_s"], ref["V_act"], ref["V_w"], ref["p_lo"], ref["p_hi"]]
        assert np.allclose(V[:, :3], Vo[:, :3], rtol=3e-2, atol=1e-12), (period, V, Vo)
        assert np.allclose(V[:, 3:], Vo[:, 3:], atol=1e-6)
        s_g, rho_g, nu_g = vb.update_ratios(s_g, rho_g, nu_g, V[:, 0], V[:, 1], V[:, 2], V[:, 3], V[:, 4], cfg)
        s_o, rho_o, nu_o = o.update_ratios(s_o, rho_o, nu_o, Vo[:, 0], Vo[:, 1], Vo[:, 2], Vo[:, 3], Vo[:, 4], **kw)
        assert s_g == pytest.approx(s_o, abs=1e-6)
        assert np.allclose(rho_g, rho_o, atol=1e-6) and np.allclose(nu_g, nu_o, rtol=1e-5)
        assert np.all(np.diff(rho_g) >= 0) and min(rho_g) >= 1.0 / N
        moved = moved or s_g < 1.0 or min(nu_g) < 1.0
        for step in range(2):
            stack.backward(rho_g[::-1], nu_g[::-1], seed=10 * period + step, variant=step)
        assert stack.device_status() == 0
    assert moved
    stack.close()


def test_bad_alive_list_is_reported_not_followed():
    """A caller's alive list with a length beyond N or an entry outside [0, N) is skipped by the kernels' own
    checks and reported through the status word."""
    vbuild.build()
    N, T, d_in, d_out = 8, 64, 128, 192
    case = inputs.LayerCase("bad", N, T, d_in, d_out, BF16, 1.0, 0.5, 0.5, 0.5)
    X, dY, W = [t.cuda() for t in inputs.make_layer(case)]
    lay = vb.Layer(N, T, d_in, d_out, BF16, vb.GEMM_TENSOR)
    dX = torch.empty(N * T, d_in, dtype=BF16, device="cuda")
    dW = torch.empty(d_out, d_in, dtype=torch.float32, device="cuda")
    alive = torch.tensor([0, 3, N + 5, -2, 6, 7, 1, 2], dtype=torch.int32, device="cuda")
    for cnt in (5, N + 3):
        c = torch.tensor([cnt], dtype=torch.int32, device="cuda")
        lay.linear_bwd_chain(X, dY, W, 0.5, 0.5, 1, dX, dW, alive_in=alive, alive_cnt_in=c)
        assert lay.device_status() == -1
    good = torch.tensor([0, 3, 6], dtype=torch.int32, device="cuda")
    lay.linear_bwd_chain(X, dY, W, 0.9, 0.5, 1, dX, dW, alive_in=good,
                         alive_cnt_in=torch.tensor([3], dtype=torch.int32, device="cuda"))
    assert lay.device_status() == 0
    s = lay.last_sampling()
    assert set(s.idxA.cpu().tolist()) <= {0, 3, 6}
    lay.close()


def test_skip_dropped_rows_leaves_them_untouched():
    """With skip_dropped_rows the rows of dX of dropped data are not written; the kept rows are the same bits."""
    vbuild.build()
    N, T, d_in, d_out = 10, 197, 320, 192
    case = inputs.LayerCase("skip", N, T, d_in, d_out, BF16, 1.0, 0.5, 0.5, 0.5)
    X, dY, W = [t.cuda() for t in inputs.make_layer(case)]
    lay = vb.Layer(N, T, d_in, d_out, BF16, vb.GEMM_TENSOR)
    ref = torch.empty(N * T, d_in, dtype=BF16, device="cuda")
    dW = torch.empty(d_out, d_in, dtype=torch.float32, device="cuda")
    kept = torch.zeros(N, dtype=torch.int32, device="cuda"); cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    lay.linear_bwd_chain(X, dY, W, 0.5, 0.5, 4, ref, dW, kept_out=kept, kept_cnt_out=cnt)
    dX = torch.full((N * T, d_in), 7.0, dtype=BF16, device="cuda")
    lay.linear_bwd_chain(X, dY, W, 0.5, 0.5, 4, dX, dW, kept_out=kept, kept_cnt_out=cnt, skip_dropped_rows=True)
    k = kept[:int(cnt.item())].cpu().numpy()
    keep = np.zeros(N, bool); keep[k] = True
    assert 0 < keep.sum() < N
    rows = torch.from_numpy(np.repeat(keep, T)).cuda()
    assert torch.equal(dX[rows], ref[rows]) and not ref[~rows].any()
    assert torch.all(dX[~rows] == 7.0)
    assert lay.device_status() == 0
    lay.close()


def test_overlapped_layers_give_the_same_bits():
    """With defer_join a layer's weight-gradient branch runs beside the next layers; results are unchanged, also when
    a pass is replayed from a CUDA graph."""
    vbuild.build()
    dev = torch.device("cuda")
    N, T, d, ffn, qkv = 8, 64, 256, 512, 384
    outs = []
    for overlap in (False, True):
        layers = []
        for block in (2, 1, 0):
            layers += make_block_layers(N, T, d, ffn, qkv, block, 1, dev)
        stack = LinearStack(layers, N, T, gemm_path=vb.GEMM_TENSOR, overlap_layers=overlap, skip_dropped_rows=True)
        L = len(layers)
        rho, nu = np.linspace(0.8, 0.4, L), np.full(L, 0.5)
        stack.backward(rho, nu, seed=5)
        torch.cuda.synchronize()
        res = [(l.dW.clone(), l.kept.clone(), l.kept_cnt.clone()) for l in layers]
        if overlap:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                stack.backward(rho, nu, seed=5)
            for l in layers:
                l.dW.zero_()
            g.replay()
            torch.cuda.synchronize()
            for l, (dW, kept, cnt) in zip(layers, res):
                assert torch.equal(l.dW, dW) and torch.equal(l.kept_cnt, cnt)
        outs.append(res)
        assert stack.device_status() == 0
        stack.close()
    for (dW0, k0, c0), (dW1, k1, c1) in zip(*outs):
        assert torch.equal(dW0, dW1) and torch.equal(c0, c1) and torch.equal(k0[:int(c0.item())], k1[:int(c1.item())])
