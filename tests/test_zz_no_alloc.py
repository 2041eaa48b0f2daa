"""br_power_static: the Power() step for callers that cannot allocate device memory (a process whose
framework owns all of HBM, a service that forbids allocation after start-up, a loop that cannot
take cudaMalloc's device-wide synchronisation).  Its scratch is a fixed array in the library's
device image instead of the handle's slab.

Checked here, through the C-ABI, on two calls in a row (the second one finds the first one's
leftovers in the shared array): the result equals what the handle-based path (br_set_state +
br_refresh_basis) produces from the same factor and basis, within the basis tolerance of the other
tests (sign-normalised max-abs 1e-3), and equals the float64 oracle's Power(F, Q) within the same
tolerance.  Odd orders are covered as well (the work area behind the k x k product must stay on a
vector-access boundary for them).  Orders beyond the fixed scratch are rejected."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL_BASIS = 1e-3


def _factor(k, seed):
    rng = np.random.default_rng(seed)
    Qe, _ = np.linalg.qr(rng.standard_normal((k, k)))
    lam = np.logspace(0, -3, k)
    F = ((Qe * lam) @ Qe.T).astype(np.float32)
    Q0, _ = np.linalg.qr(rng.standard_normal((k, k)))
    return F, Q0.astype(np.float32)


@pytest.mark.parametrize("k", [200, 129, 201])      # several panels, the last one ragged; odd orders
def test_static_scratch_power_matches_handle_path_twice(k):
    import torch
    import paper_2602_03515_b200 as br
    from oracle import br_oracle as O
    from workloads import LayerSpec
    from tests.parity_util import basis_err
    w = torch.zeros(k, 16, device="cuda")
    opt = br.BasisRotation([LayerSpec("W", k, 16, br.BR_GEOM_BILATERAL, br.BR_SRC_SECOND, 0)], [w],
                           grad_dtype="f32", gemm_prec=br.BR_GEMM_FP32, freq=10 ** 6)
    try:
        assert opt.step([torch.randn(k, 16, device="cuda") * 0.01], 0) == br.BR_OK
        flag = torch.full((1,), 7, dtype=torch.int32, device="cuda")
        for call, seed in enumerate((21, 22)):
            F, Q0 = _factor(k, seed)
            # existing entry points
            opt.set_state(0, br.BR_BUF_L, torch.from_numpy(F))
            opt.set_state(0, br.BR_BUF_U, torch.from_numpy(Q0))
            opt.refresh_basis(0)
            assert opt.sync_status() == br.BR_OK
            want = opt.get_state(0, br.BR_BUF_U).numpy().astype(np.float64)
            # the entry point that allocates nothing
            Fd, Qd = torch.from_numpy(F).cuda(), torch.from_numpy(Q0).cuda()
            torch.cuda.synchronize()
            st = br.br_power_static(torch.cuda.current_stream().cuda_stream, Fd.data_ptr(), Qd.data_ptr(), k,
                                    flag.data_ptr())
            assert st == br.BR_OK
            torch.cuda.synchronize()
            got = Qd.cpu().numpy().astype(np.float64)
            assert int(flag.item()) == 0
            assert np.all(np.isfinite(got))
            assert basis_err(got, want) <= TOL_BASIS, (call, basis_err(got, want))
            ref, deficient = O.power(F.astype(np.float64), Q0.astype(np.float64))
            assert not deficient
            assert basis_err(got, ref) <= TOL_BASIS, (call, basis_err(got, ref))
            assert np.max(np.abs(got.T @ got - np.eye(k))) < 1e-5
    finally:
        opt.close()


def test_static_scratch_rejects_orders_beyond_its_array():
    import torch
    import paper_2602_03515_b200 as br
    x = torch.zeros(8, 8, device="cuda")
    with pytest.raises(br.BrError) as e:
        br.br_power_static(0, x.data_ptr(), x.data_ptr(), 513)
    assert e.value.status == br.BR_ERR_SHAPE
    with pytest.raises(br.BrError) as e:
        br.br_power_static(0, 0, x.data_ptr(), 8)
    assert e.value.status == br.BR_ERR_INVALID
