"""Failure handling of the library, exercised without faulting, trapping or hanging the GPU:

* a bounded device-side wait that nothing satisfies gives up after its limit, reports BR_ERR_TIMEOUT
  through the status word, and leaves the context and the handle usable;
* an allocator that returns NULL gives BR_ERR_OOM with the byte count, and nothing is leaked;
* a failed enqueue in the middle of br_step / br_refresh_basis (injected on the host: the CUDA call
  is not issued and reports a launch failure) returns BR_ERR_CUDA with the integer state as it was
  before the call, and the handle can still be read and destroyed.
"""
import ctypes as C

import numpy as np
import pytest

from workloads import LayerSpec
from workloads.configs import GEOM_BI, GEOM_UNI, SRC_FIRST, SRC_SECOND

pytestmark = pytest.mark.gpu


def _handle(br, torch, prec, tau=1, freq=2):
    specs = [LayerSpec("a", 128, 136, GEOM_BI, SRC_SECOND, tau), LayerSpec("b", 72, 264, GEOM_UNI, SRC_FIRST, tau)]
    ws = [torch.randn(s.m, s.n, device="cuda") * 0.02 for s in specs]
    dt = "bf16" if prec == br.BR_GEMM_BF16 else "f32"
    opt = br.BasisRotation(specs, ws, grad_dtype=dt, gemm_prec=prec, freq=freq)
    tdt = torch.bfloat16 if dt == "bf16" else torch.float32
    grads = lambda: [(torch.randn(s.m, s.n, device="cuda") * 0.01).to(tdt) for s in specs]
    return opt, ws, grads


def test_bounded_wait_runs_out_and_reports_timeout():
    import torch
    import paper_2602_03515_b200 as br
    opt, ws, grads = _handle(br, torch, br.BR_GEMM_BF16)
    try:
        for _ in range(3):
            opt.step(grads(), 1)
        assert opt.sync_status() == br.BR_OK
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        br.br_debug_wait_timeout(opt.handle, 1_000_000)          # 1 ms on a barrier nobody arrives on
        t1.record()
        with pytest.raises(br.BrError) as e:
            opt.sync_status()
        assert e.value.status == br.BR_ERR_TIMEOUT
        assert 0.9 <= t0.elapsed_time(t1) < 100.0                # it waited its limit, and it ended
        # the status word is sticky: contraction launches of later steps return at once
        before = [w.clone() for w in ws]
        c0 = opt.counters(0)
        opt.step(grads(), 1)
        torch.cuda.synchronize()
        for a, b in zip(ws, before):
            assert torch.equal(a, b)
        with pytest.raises(br.BrError) as e:
            opt.sync_status()
        assert e.value.status == br.BR_ERR_TIMEOUT
        assert opt.counters(0)["calls"] == c0["calls"] + 1
        assert torch.isfinite(opt.get_state(0, br.BR_BUF_U)).all()   # the handle can still be read ...
        with pytest.raises(br.BrError):
            br.br_debug_wait_timeout(opt.handle, 10)                 # (limit below 1 us: rejected on the host)
    finally:
        opt.close()                                                  # ... and destroyed
    # the context is intact: a fresh handle works
    opt2, _, grads2 = _handle(br, torch, br.BR_GEMM_BF16)
    try:
        for _ in range(3):
            opt2.step(grads2(), 1)
        assert opt2.sync_status() == br.BR_OK
    finally:
        opt2.close()


def test_allocator_returning_null_is_out_of_memory_without_leak():
    import torch
    import paper_2602_03515_b200 as br
    from paper_2602_03515_b200 import binding as B
    calls = {"alloc": [], "free": []}
    refuse = {"on": True}
    blocks = {}

    def alloc(nbytes, _ctx):
        calls["alloc"].append(int(nbytes))
        if refuse["on"]:
            return None
        t = torch.empty(int(nbytes), dtype=torch.uint8, device="cuda")
        blocks[t.data_ptr()] = t
        return t.data_ptr()

    def free(ptr, _ctx):
        calls["free"].append(ptr)
        blocks.pop(ptr, None)

    cb = (B._ALLOC_FN(alloc), B._FREE_FN(free))
    allocator = B.BrAllocator(cb[0], cb[1], None)
    w = torch.zeros(128, 136, device="cuda")
    desc = br.BrLayerDesc(m=128, n=136, geom=GEOM_BI, src=SRC_SECOND, grad_dtype=br.BR_BF16, tau_max=1, freq=0, reserved=0,
                          weight=w.data_ptr())
    hp = br.BrHparams(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, beta_factor=-1.0, freq=2,
                      power_iters=1, accum=0, gemm_prec=br.BR_GEMM_BF16, flags=0, clip_norm=0.0, scratch_limit_bytes=0)
    want, _ = br.br_state_bytes([desc], hp)
    with pytest.raises(br.BrError) as e:
        br.br_create([desc], hp, 0, 0, allocator)
    assert e.value.status == br.BR_ERR_OOM
    assert len(calls["alloc"]) == 1 and calls["free"] == []              # asked once, nothing to give back
    assert str(calls["alloc"][0]) in br.br_last_error(None)              # the byte count is in the message
    assert abs(calls["alloc"][0] - want) <= 256                          # and it is what br_state_bytes announces
    # the same allocator, now serving: create works; a temporary it refuses later is BR_ERR_OOM too and
    # leaves the handle usable; destroy returns the one block
    refuse["on"] = False
    h = br.br_create([desc], hp, 0, 0, allocator)
    try:
        g = (torch.randn(128, 136, device="cuda") * 0.01).to(torch.bfloat16)
        for _ in range(3):
            assert br.br_step(h, [g.data_ptr()], 1) >= 0
        out = torch.empty(128, 136)
        refuse["on"] = True
        with pytest.raises(br.BrError) as e:
            br.br_get_state(h, 0, br.BR_BUF_M, out.data_ptr(), out.numel() * 4)      # needs 8 m n bytes of temporary memory
        assert e.value.status == br.BR_ERR_OOM
        refuse["on"] = False
        br.br_get_state(h, 0, br.BR_BUF_M, out.data_ptr(), out.numel() * 4)
        assert torch.isfinite(out).all() and br.br_sync_status(h) == br.BR_OK
    finally:
        br.br_destroy(h)
    assert len(calls["free"]) == len(calls["alloc"]) - 2 and not blocks     # two refused requests, the rest returned


@pytest.mark.parametrize("prec", ["fp32", "bf16"])
def test_failed_enqueue_leaves_the_integer_state_untouched(prec):
    """Every position of the injected failure over a whole step that contains a refresh (fork and join
    of the refresh lanes, side-stream ring copies, re-expression of the rotated momentum)."""
    import torch
    import paper_2602_03515_b200 as br
    gp = br.BR_GEMM_BF16 if prec == "bf16" else br.BR_GEMM_FP32
    hit = 0
    for countdown in list(range(0, 40)) + [60, 90, 130, 200]:
        opt, ws, grads = _handle(br, torch, gp, tau=1, freq=2)
        try:
            for _ in range(2):                       # warm-up call + update t = 1; the next update (t = 2) refreshes
                opt.step(grads(), 1)
            assert opt.sync_status() == br.BR_OK
            c_before = [opt.counters(i) for i in range(2)]
            br.br_debug_inject(opt.handle, br.BR_INJECT_LAUNCH_FAILURE, countdown)
            try:
                opt.step(grads(), 1)
                failed = False
            except br.BrError as e:
                assert e.status == br.BR_ERR_CUDA
                failed = True
            br.br_debug_inject(opt.handle, br.BR_INJECT_NONE, 0)
            torch.cuda.synchronize()
            if failed:
                hit += 1
                assert [opt.counters(i) for i in range(2)] == c_before
                assert torch.isfinite(opt.get_state(0, br.BR_BUF_V2)).all()      # still readable
            else:
                assert opt.counters(0)["t"] == c_before[0]["t"] + 1 and opt.counters(0)["refresh_count"] == 1
        finally:
            opt.close()                              # and destroyable, with the lanes joined
    assert hit >= 20                                 # the step issues far more than 20 CUDA calls
    torch.cuda.synchronize()


def test_failed_enqueue_inside_forced_refresh():
    import torch
    import paper_2602_03515_b200 as br
    for countdown in (0, 2, 5, 9, 14, 20):
        opt, ws, grads = _handle(br, torch, br.BR_GEMM_BF16, tau=0, freq=100)
        try:
            opt.step(grads(), 0)
            c_before = opt.counters(0)
            br.br_debug_inject(opt.handle, br.BR_INJECT_LAUNCH_FAILURE, countdown)
            with pytest.raises(br.BrError) as e:
                opt.refresh_basis(-1)
            assert e.value.status == br.BR_ERR_CUDA
            br.br_debug_inject(opt.handle, br.BR_INJECT_NONE, 0)
            assert opt.counters(0) == c_before
        finally:
            opt.close()
    torch.cuda.synchronize()


@pytest.mark.parametrize("prec", ["fp32", "bf16"])
def test_debug_canaries_stay_intact_and_catch_an_overrun(prec):
    """BR_FLAG_DEBUG_CANARY puts guard words behind every piece of the handle's memory.  A run through
    steps and refreshes (factor products, rotations, refresh lanes, tensor-core scratch) leaves all of
    them intact; a word overwritten from the host side, inside the test's own allocation, is reported
    with its position.  A handle without the flag has no guards to check."""
    import torch
    import paper_2602_03515_b200 as br
    gp = br.BR_GEMM_BF16 if prec == "bf16" else br.BR_GEMM_FP32
    specs = [LayerSpec("a", 128, 136, GEOM_BI, SRC_SECOND, 2), LayerSpec("b", 72, 264, GEOM_UNI, SRC_FIRST, 1),
             LayerSpec("c", 40, 24, GEOM_BI, SRC_SECOND, 0)]
    ws = [torch.randn(s.m, s.n, device="cuda") * 0.02 for s in specs]
    dt = "bf16" if prec == "bf16" else "f32"
    tdt = torch.bfloat16 if prec == "bf16" else torch.float32
    opt = br.BasisRotation(specs, ws, grad_dtype=dt, gemm_prec=gp, freq=3, flags=br.BR_FLAG_DEBUG_CANARY)
    try:
        for _ in range(9):
            opt.step([(torch.randn(s.m, s.n, device="cuda") * 0.01).to(tdt) for s in specs], -1)
        opt.refresh_basis(-1)
        assert opt.sync_status() == br.BR_OK
        assert br.br_debug_check_canaries(opt.handle) == br.BR_OK
        # the slab is the one block the torch-backed allocator handed out: find a guard in it and damage it
        (slab,) = opt._blocks.values()
        host = slab.cpu().numpy()
        word = np.frombuffer(host.tobytes(), dtype=np.uint32)
        runs = np.flatnonzero(word == 0xC5C5C5C5)
        assert len(runs) >= 64 * 10                       # dozens of guards of 64 words each
        slab[int(runs[100]) * 4] = 0                      # one byte of one guard
        torch.cuda.synchronize()
        with pytest.raises(br.BrError) as e:
            br.br_debug_check_canaries(opt.handle)
        assert e.value.status == br.BR_ERR_STATE and "canary" in str(e.value)
    finally:
        opt.close()
    plain = br.BasisRotation(specs[2:], ws[2:], grad_dtype=dt, gemm_prec=gp)
    try:
        with pytest.raises(br.BrError) as e:
            br.br_debug_check_canaries(plain.handle)
        assert e.value.status == br.BR_ERR_STATE
    finally:
        plain.close()
