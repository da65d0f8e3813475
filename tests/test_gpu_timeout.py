"""The exit path behind LBP_ERR_TIMEOUT, exercised without faulting a device.

Every wait inside the persistent products kernel is bounded.  The test hook
lbp_test_stall_products makes the TMA producers issue nothing, so that no copy
is in flight and the tensor-core issuer and the epilogue warps run into their
limits (about a second).  The kernel must then report LBP_ERR_TIMEOUT through
the status block, give its tensor memory back and return; the context stays
usable and the next ordinary call on the same workspace passes parity.
"""
import pytest
import torch

import paper_2309_15275_b200 as lbp
import synth
from oracle import lbp_oracle as O

pytestmark = pytest.mark.gpu

LBP_ERR_TIMEOUT = 10


def f64(t):
    return t.detach().cpu().to(torch.float64).numpy()


# Cin = 256 takes the CTA-pair kernel, Cin = 64 the one-CTA kernel
@pytest.mark.parametrize("Cin,Cout", [(256, 128), (64, 64)])
def test_expired_wait_is_reported_and_the_next_call_is_clean(Cin, Cout):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    k, r = 8, 4
    case = synth.LayerCase(3, "tiny_stall", 2, 16, 16, Cin, Cout, k, (r,), "bf16",
                           ("normal", 1.0), ("normal", 0.01), 11)
    x, gy, w = synth.make_layer_inputs(case)
    bases = lbp.lbp_select_bases(k, lbp.SEL_PREFIX, r)
    xd, gd, wd = x.to(dev), gy.to(dev), w.to(dev)
    ws = lbp.alloc_workspace(xd, gd, k, r)
    ws.zero_()
    lbp.lbp_test_stall_products(True)
    try:
        lbp.lbp_backward(xd, gd, wd, k, bases, ws=ws)
    finally:
        lbp.lbp_test_stall_products(False)
    assert lbp.lbp_poll_status(ws) == LBP_ERR_TIMEOUT
    assert lbp.lbp_poll_status(ws) == 0            # reading the status clears it
    gx, gw = lbp.lbp_backward(xd, gd, wd, k, bases, ws=ws)
    assert lbp.lbp_poll_status(ws) == 0
    ox, ow = O.backward_lowrank(f64(x), f64(gy), f64(w), k, bases)
    assert O.rel_fro(f64(gx), ox) <= 2e-2 and O.rel_fro(f64(gw), ow) <= 2e-2


def test_expired_wait_in_the_projection_kernel():
    # the same for the tcgen05 projection kernel: no box is fetched, the tensor-core
    # issuer and the epilogue warps give up, the status says so, the next call is clean
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    k, r = 8, 6
    t = synth.make_tensor((2, 16, 24, 256), ("normal", 1.0), "bf16", case_key=2500).to(dev)
    bases = lbp.lbp_select_bases(k, lbp.SEL_PREFIX, r)
    ws = torch.zeros(lbp.lbp_status_bytes(), dtype=torch.uint8, device=dev)
    lbp.lbp_test_stall_products(True, projection=True)
    try:
        lbp.lbp_project(t, k, bases, ws=ws)
    finally:
        lbp.lbp_test_stall_products(False)
    assert lbp.lbp_poll_status(ws) == LBP_ERR_TIMEOUT
    assert lbp.lbp_poll_status(ws) == 0
    got = lbp.lbp_project(t, k, bases, ws=ws)
    assert lbp.lbp_poll_status(ws) == 0
    assert O.rel_fro(f64(got), O.project(f64(t), k, bases)) <= 2e-2
