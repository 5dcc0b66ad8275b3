"""The C-ABI library builds, loads and exports what include/vcas.h declares; host-only entry
points are checked against the oracle.  No GPU needed."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import vcas_oracle as o
from paper_2402_17227_b200 import binding as vb
from paper_2402_17227_b200 import build as vbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    vbuild.build()
    return vb.lib()


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            text = open(os.path.join(inc, f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\bint\s+(vcas_\w+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"vcas_linear_bwd", "vcas_score", "vcas_variance_probe", "vcas_update_ratios"} <= names
    for n in names:
        assert hasattr(lib, n), n
    assert names == set(vb.EXPORTS)          # the binding covers the whole header
    assert lib.vcas_version() >= 100


def test_default_config_is_the_papers(lib, golden_dir):
    consts = dict(l.split() for l in open(os.path.join(golden_dir, "paper_constants.txt"))
                  if l.strip() and not l.startswith("#"))
    cfg = vb.default_config()
    assert cfg.tau_act == pytest.approx(float(consts["tau"])) and cfg.tau_w == pytest.approx(float(consts["tau"]))
    assert cfg.alpha == pytest.approx(float(consts["alpha"])) and cfg.beta == pytest.approx(float(consts["beta"]))
    assert cfg.M == int(consts["M"])


def test_bad_arguments_return_codes(lib):
    assert lib.vcas_default_config(None) == -1
    h = C.c_void_p(None)
    assert lib.vcas_create(C.byref(h), None, None) == -1
    bad = vb.LayerDesc(4, 4, 12, 16, vb.DTYPE_F32, 0)         # d_in not a multiple of 8
    assert lib.vcas_create(C.byref(h), C.byref(bad), None) == -2
    bad = vb.LayerDesc(4, 4, 16, 16, 7, 0)
    assert lib.vcas_create(C.byref(h), C.byref(bad), None) == -3
    bad = vb.LayerDesc(4, 4, 16, 16, vb.DTYPE_F32, vb.GEMM_TENSOR)   # tensor path needs bf16, multiples of 64
    assert lib.vcas_create(C.byref(h), C.byref(bad), None) == -2
    assert lib.vcas_destroy(None) == -1
    assert lib.vcas_linear_bwd(None, None, None, None, C.c_float(0.5), C.c_float(0.5), C.c_uint64(0), None, None,
                               None) == -1
    assert lib.vcas_update_ratios(None, 1, None, None, None, None, None, None) == -1


@pytest.mark.parametrize("seed", range(8))
def test_update_ratios_matches_oracle(lib, seed):
    r = np.random.default_rng(seed)
    L = int(r.integers(1, 30))
    f32 = lambda x: np.asarray(x, dtype=np.float32)
    V_s, V_act, V_w = f32(r.random(L) * 10), f32(r.random(L) * 0.5), f32(r.random(L) * 0.5)
    p_lo, p_hi = f32(r.random(L)), f32(r.random(L))
    rho, nu = f32(r.random(L)), f32(r.uniform(0.05, 1.0, L))
    s = float(f32(r.uniform(0, 1)))
    cfg = vb.default_config()
    cfg.nu_min = 0.1
    cfg.rho_min = 0.05
    s2, rho2, nu2 = vb.update_ratios(s, rho, nu, V_s, V_act, V_w, p_lo, p_hi, cfg)
    es, erho, enu = o.update_ratios(s, rho.astype(np.float64), nu.astype(np.float64), V_s, V_act, V_w, p_lo, p_hi,
                                    tau_act=float(cfg.tau_act), tau_w=float(cfg.tau_w), alpha=float(cfg.alpha),
                                    beta=float(cfg.beta), rho_min=float(cfg.rho_min), nu_min=float(cfg.nu_min))
    assert s2 == pytest.approx(es, abs=1e-7)
    assert np.allclose(rho2, erho, rtol=1e-6) and np.allclose(nu2, enu, rtol=1e-6)
    assert np.all(np.diff(rho2) >= 0)


def test_update_ratios_sign_zero_and_clipping(lib):
    cfg = vb.default_config()
    cfg.tau_act = 0.25          # exactly representable, so that equality is exact
    cfg.tau_w = 0.25
    # V_act == tau V_s exactly: sign(0) = +1 -> s goes up, p_hi chosen
    s, rho, nu = vb.update_ratios(0.5, [1.0], [0.5], [4.0], [1.0], [1.0], [0.25], [0.75], cfg)
    assert s == pytest.approx(0.51) and rho == [0.75] and nu[0] == pytest.approx(0.5 / 0.95)
    s, _, nu = vb.update_ratios(1.0, [1.0], [1.0], [4.0], [2.0], [2.0], [0.25], [0.75], cfg)
    assert s == 1.0 and nu == [1.0]
    s, _, _ = vb.update_ratios(0.004, [1.0], [1.0], [40.0], [0.0], [0.0], [0.25], [0.75], cfg)
    assert s == 0.0
