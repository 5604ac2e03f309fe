"""Error paths of the C ABI on the device: a bounded wait that runs out (in the safe, self-releasing form), a
workspace that is too small, and a status word that is already raised when an optimisation loop starts."""
import ctypes

import numpy as np
import pytest

import cafeq_synth as syn
from parity_utils import f32_dev, to_dev

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cq():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2511_19705_b200 as m
    m.lib()
    return m


def test_bounded_wait_runs_out_and_reports_timeout(cq):
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    result = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    rc = cq.lib().cafeq_debug_wait_probe(ctypes.c_ulonglong(2000), cq._p(status), cq._p(result), cq._stream())
    assert rc == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 7                      # CAFEQ_ERR_TIMEOUT
    assert result.tolist() == [1, 1]                    # the first wait gave up, the second (after the arrival) succeeded
    assert cq.status_string(7) == "bounded device wait expired"
    # the context is intact: an ordinary call runs afterwards
    Wd = to_dev(syn.weight_student_t(64, 256, 1))
    codes, scales = cq.cafeq_rtn(Wd, None, bits=4, group=128)
    torch.cuda.synchronize()
    assert int(codes.abs().max().item()) == 7


def test_too_small_workspace_is_refused_before_any_launch(cq):
    d_out, d_in, k = 256, 512, 128
    Wd = to_dev(syn.weight_student_t(d_out, d_in, 2))
    M = f32_dev(syn.haar_blocks(d_in // k, k, 3))
    d = cq.make_desc(d_out, d_in, 4, 128, k, cq.AXIS_IN, 0, 1, d_in)
    need = cq.workspace_size(d)
    losses = torch.full((4,), -5.0, dtype=torch.float32, device="cuda")
    grad = torch.full_like(M, -5.0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(need // 4, dtype=torch.uint8, device="cuda")
    n0 = cq.launch_count()
    rc = cq.lib().cafeq_proxy_loss_fwd_bwd(ctypes.byref(d), cq._p(Wd), cq._p(M), cq._p(None), cq._p(None), ctypes.c_int(0),
                                           ctypes.c_int(cq.LOSS_SURROGATE), ctypes.c_float(0.0), ctypes.c_int(0),
                                           cq._p(losses), cq._p(grad), cq._p(None), cq._p(status), cq._p(ws), ctypes.c_size_t(ws.numel()),
                                           cq._stream())
    torch.cuda.synchronize()
    assert rc == 3                                       # CAFEQ_ERR_WORKSPACE
    assert cq.launch_count() == n0                       # nothing was enqueued
    assert float(losses.min().item()) == -5.0 and float(grad.max().item()) == -5.0   # outputs untouched
    # a misaligned workspace is refused the same way
    big = torch.empty(need + 512, dtype=torch.uint8, device="cuda")
    rc = cq.lib().cafeq_proxy_loss_fwd_bwd(ctypes.byref(d), cq._p(Wd), cq._p(M), cq._p(None), cq._p(None), ctypes.c_int(0),
                                           ctypes.c_int(cq.LOSS_SURROGATE), ctypes.c_float(0.0), ctypes.c_int(0),
                                           cq._p(losses), cq._p(grad), cq._p(None), cq._p(status), ctypes.c_void_p(big.data_ptr() + 8),
                                           ctypes.c_size_t(need), cq._stream())
    assert rc == 3


def test_lean_workspace_runs_the_same_optimisation(cq):
    """The configuration-specific (lean) workspace of the Eq. 4 loop is a small fraction of the general one and
    gives the same parameters; asking it for the quantised loss is refused."""
    d_out, d_in, k = 4000, 512, 256
    Wd = to_dev(syn.weight_student_t(d_out, d_in, 8, 2, 10.0))
    M0 = syn.perturbed_blocks(d_in // k, k, 4, 0.05)
    d = cq.make_desc(d_out, d_in, 3, 128, k, cq.AXIS_IN, 0, 1, d_in)
    g0 = cq.cafeq_proxy_loss_fwd_bwd(Wd, f32_dev(M0), bits=3, group=128)["gradM"]
    lr = float(1e-3 / g0.abs().max().item())
    cfg = cq.make_cfg(loss_kind=cq.LOSS_SURROGATE, optimizer=cq.OPT_GD, lr=lr, steps=3)
    full, lean = cq.workspace_size(d), cq.workspace_size(d, None, cfg)
    assert lean < full // 3
    outs = []
    for nbytes in (full, lean):
        M = f32_dev(M0)
        hist = torch.zeros((3, 2), dtype=torch.float32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        rc = cq.lib().cafeq_optimize_single(ctypes.byref(d), cq._p(Wd), cq._p(M), cq._p(None), ctypes.byref(cfg), cq._p(hist),
                                            cq._p(status), cq._p(ws), ctypes.c_size_t(nbytes), cq._stream())
        torch.cuda.synchronize()
        assert rc == 0 and int(status.item()) == 0
        outs.append((M.cpu().numpy(), hist.cpu().numpy()))
    # (the same kernels; the gradient's floating-point atomics may add in another order)
    assert np.allclose(outs[0][0], outs[1][0], rtol=0, atol=1e-6) and np.allclose(outs[0][1][:, 0], outs[1][1][:, 0], rtol=1e-5)
    cfg_eval = cq.make_cfg(loss_kind=cq.LOSS_SURROGATE, optimizer=cq.OPT_GD, lr=lr, steps=1, eval_every=1)
    M = f32_dev(M0)
    hist = torch.zeros((1, 2), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(lean, dtype=torch.uint8, device="cuda")
    rc = cq.lib().cafeq_optimize_single(ctypes.byref(d), cq._p(Wd), cq._p(M), cq._p(None), ctypes.byref(cfg_eval), cq._p(hist),
                                        cq._p(status), cq._p(ws), ctypes.c_size_t(lean), cq._stream())
    assert rc == 3


def test_raised_status_stops_the_remaining_steps(cq):
    d_out, d_in, k = 256, 512, 128
    Wd = to_dev(syn.weight_student_t(d_out, d_in, 9))
    M0 = syn.perturbed_blocks(d_in // k, k, 5, 0.05)
    M = f32_dev(M0)
    d = cq.make_desc(d_out, d_in, 4, 128, k, cq.AXIS_IN, 0, 1, d_in)
    cfg = cq.make_cfg(loss_kind=cq.LOSS_SURROGATE, optimizer=cq.OPT_GD, lr=1e-2, steps=4)
    hist = torch.full((4, 2), -3.0, dtype=torch.float32, device="cuda")
    status = torch.full((1,), 6, dtype=torch.int32, device="cuda")     # a non-finite value was met earlier
    ws = torch.empty(cq.workspace_size(d), dtype=torch.uint8, device="cuda")
    rc = cq.lib().cafeq_optimize_single(ctypes.byref(d), cq._p(Wd), cq._p(M), cq._p(None), ctypes.byref(cfg), cq._p(hist),
                                        cq._p(status), cq._p(ws), ctypes.c_size_t(ws.numel()), cq._stream())
    torch.cuda.synchronize()
    assert rc == 0 and int(status.item()) == 6           # first error wins
    assert np.array_equal(M.cpu().numpy(), M0)           # no step changed the parameters
    # a singular block raises the status on the device and the later steps leave the parameters alone
    Ms = M0.copy()
    Ms[1] = 0.0
    M = f32_dev(Ms)
    status.zero_()
    rc = cq.lib().cafeq_optimize_single(ctypes.byref(d), cq._p(Wd), cq._p(M), cq._p(None), ctypes.byref(cfg), cq._p(hist),
                                        cq._p(status), cq._p(ws), ctypes.c_size_t(ws.numel()), cq._stream())
    torch.cuda.synchronize()
    assert rc == 0 and int(status.item()) in (5, 6)      # singular block (or the non-finite values it produced)
    assert np.array_equal(M.cpu().numpy(), Ms)
