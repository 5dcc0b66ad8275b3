"""Failure detection on the device: a wait inside a product kernel that can never be satisfied must run out,
be reported as VCAS_ERR_TIMEOUT, leave the GPU context intact, and leave the handle usable.  The wait is made
to run out with the library's test hook (the first CTA does not issue the loads of its first k-block; nothing
faults and no loop is unbounded: every wait gives up after the limit set here, two milliseconds)."""
import pytest
import torch

from paper_2402_17227_b200 import binding as vb
from paper_2402_17227_b200 import build as vbuild
from paper_2402_17227_b200 import inputs

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


# tile widths / slices / tile heights that select the three instances of the product kernel:
# tiles in CTA order, the sliced contraction, and (more tiles than SMs) the device-wide work counter
@pytest.mark.parametrize("shape,tuning", [((6, 160, 192, 256), (0, 0, 0, 0, 0)),
                                          ((6, 160, 192, 256), (256, 256, 3, 3, 1)),
                                          ((48, 512, 512, 256), (256, 256, 1, 1, 2))])
def test_wait_runs_out_and_handle_recovers(shape, tuning):
    vbuild.build()
    N, T, d_in, d_out = shape
    case = inputs.LayerCase("g", N, T, d_in, d_out, BF16, 1.0, 0.5, 0.5, 0.5)
    X, dY, W = [t.cuda() for t in inputs.make_layer(case)]
    clean = vb.Layer(N, T, d_in, d_out, BF16, vb.GEMM_TENSOR)
    clean.set_tuning(*tuning)
    ref_dX, ref_dW = clean.linear_bwd(X, dY, W, 0.6, 0.5, 3)
    ref_dXd, ref_dWd = clean.dense_bwd(X, dY, W)
    assert clean.device_status() == 0
    layer = vb.Layer(N, T, d_in, d_out, BF16, vb.GEMM_TENSOR)
    layer.set_tuning(*tuning)
    layer.set_wait_limit(2_000_000, stall_once=True)
    layer.linear_bwd(X, dY, W, 0.6, 0.5, 3)            # returns: the call only enqueues
    assert layer.device_status() == -6                  # VCAS_ERR_TIMEOUT, read after a device synchronise
    assert layer.device_status() == 0                   # the word is cleared by reading it
    layer.dense_bwd(X, dY, W)
    assert layer.device_status() == -6
    # the context is alive and the handle works again: bit-identical to a handle that never gave up
    layer.set_wait_limit(2_000_000_000, stall_once=False)
    for _ in range(2):
        dX, dW = layer.linear_bwd(X, dY, W, 0.6, 0.5, 3)
        assert torch.equal(dX, ref_dX) and torch.equal(dW, ref_dW)
        dXd, dWd = layer.dense_bwd(X, dY, W)
        assert torch.equal(dXd, ref_dXd) and torch.equal(dWd, ref_dWd)
    assert layer.device_status() == 0
    layer.close(); clean.close()
