"""lbp_backward_static: the entry point for callers that cannot allocate.

Some users of the library only ever hold input and output buffers: a server that
gave all device memory to its own pool and forbids cudaMalloc afterwards, a
plug-in inside a host framework, code on a path where allocating is not allowed.
For them the library carries its own fixed scratch array.  This test calls that
entry point through the C ABI twice in a row (the array is shared between calls
and keeps the previous call's contents) and checks each result against
lbp_backward with a caller-provided workspace.

The file sorts last so that a stop-at-first-failure run has already executed
every other test before this one.
"""
import pytest
import torch

import paper_2309_15275_b200 as lbp
import synth
from oracle import lbp_oracle as O

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_caller_workspace_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    k = 8
    # two different layers and ranks back to back: the second call finds the
    # first call's data in the shared scratch and must not be affected by it
    runs = [(synth.config_cases(3)[1], 8, 8), (synth.config_cases(2)[0], 1, 6)]
    for case, batch, r in runs:
        x, gy, w = (t.to(dev) for t in synth.make_layer_inputs(case, batch=batch))
        bases = lbp.lbp_select_bases(k, lbp.SEL_PREFIX, r)
        need = lbp.lbp_workspace_bytes(batch, case.H, case.W, case.Cin, case.Cout, k,
                                       lbp.LBP_BF16, lbp.LBP_F32, r)
        assert 0 < need <= lbp.STATIC_SCRATCH_BYTES
        want_gx, want_gw = lbp.lbp_backward(x, gy, w, k, bases)
        g_x = torch.empty_like(x)
        g_W = torch.empty((case.Cout, case.Cin), dtype=torch.float32, device=dev)
        lbp.lbp_backward_static(x, gy, w, k, bases, g_x=g_x, g_W=g_W)
        torch.cuda.synchronize()
        # same kernels, same tile plan, same inputs: the library is deterministic,
        # so the two entry points agree bit for bit
        assert torch.equal(g_x, want_gx)
        assert torch.equal(g_W, want_gw)
        ox, ow = O.backward_lowrank(x.cpu().double().numpy(), gy.cpu().double().numpy(),
                                    w.cpu().double().numpy(), k, bases)
        assert O.rel_fro(g_x.cpu().double().numpy(), ox) <= 2e-2
        assert O.rel_fro(g_W.cpu().double().numpy(), ow) <= 2e-2


def test_static_scratch_rejects_layers_beyond_its_size():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    case = synth.config_cases(3)[2]          # 768 -> 3072 at B = 128 needs far more than 32 MiB
    assert lbp.lbp_workspace_bytes(case.B, case.H, case.W, case.Cin, case.Cout, 8,
                                   lbp.LBP_BF16, lbp.LBP_F32, 8) > lbp.STATIC_SCRATCH_BYTES
    x = torch.zeros((case.B, case.H, case.W, case.Cin), dtype=torch.bfloat16, device=dev)
    gy = torch.zeros((case.B, case.H, case.W, case.Cout), dtype=torch.bfloat16, device=dev)
    w = torch.zeros((case.Cout, case.Cin), dtype=torch.bfloat16, device=dev)
    g_x = torch.full_like(x, 3.0)
    g_W = torch.full((case.Cout, case.Cin), 3.0, dtype=torch.float32, device=dev)
    with pytest.raises(lbp.LbpError) as e:
        lbp.lbp_backward_static(x, gy, w, 8, lbp.lbp_select_bases(8, lbp.SEL_PREFIX, 8),
                                g_x=g_x, g_W=g_W)
    assert e.value.status == 7
    torch.cuda.synchronize()
    assert torch.all(g_W == 3.0) and torch.all(g_x == 3.0)    # nothing was enqueued


def test_static_scratch_checks_arguments_before_it_enqueues_anything():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    x = torch.zeros((1, 8, 8, 64), dtype=torch.bfloat16, device=dev)
    gy = torch.zeros((1, 8, 8, 64), dtype=torch.bfloat16, device=dev)
    w = torch.zeros((64, 64), dtype=torch.bfloat16, device=dev)
    g_x = torch.full_like(x, 3.0)
    g_W = torch.full((64, 64), 3.0, dtype=torch.float32, device=dev)
    # a duplicate basis and an index outside the order: refused like lbp_backward refuses them
    for bases in ([(0, 0), (0, 0)], [(0, 8)]):
        with pytest.raises(lbp.LbpError) as e:
            lbp.lbp_backward_static(x, gy, w, 8, bases, g_x=g_x, g_W=g_W)
        assert e.value.status == 4
    with pytest.raises(lbp.LbpError) as e:      # g_W not 16-byte aligned
        lbp.lbp_backward_static(x, gy, w, 8, [(0, 0)], g_x=g_x,
                                g_W=torch.full((64 * 64 + 1,), 3.0, device=dev)[1:].view(64, 64))
    assert e.value.status == 6
    torch.cuda.synchronize()
    assert torch.all(g_W == 3.0) and torch.all(g_x == 3.0)
    # and the array still serves a valid call afterwards
    lbp.lbp_backward_static(x, gy, w, 8, [(0, 0)], g_x=g_x, g_W=g_W)
    torch.cuda.synchronize()
    assert torch.all(g_W == 0.0) and torch.all(g_x == 0.0)
