"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every symbol that
include/br.h declares, validates on the host, and reproduces the memory table of App. H."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def br():
    import __graft_entry__ as ge
    ge.build()
    import paper_2602_03515_b200 as br
    br.load_library()
    return br


def test_exports_every_declared_symbol(br):
    hdr = open(os.path.join(ROOT, "include", "br.h")).read()
    names = set(re.findall(r"BR_API\s+[\w\s\*]+?\b(br_\w+)\s*\(", hdr))
    assert {"br_create", "br_step", "br_refresh_basis", "br_destroy"} <= names
    lib = br.load_library()
    for n in sorted(names):
        assert hasattr(lib, n), n


def _hp(br, **kw):
    d = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, beta_factor=-1.0, freq=10,
             power_iters=1, accum=0, gemm_prec=br.BR_GEMM_FP32, flags=0, clip_norm=0.0, scratch_limit_bytes=0)
    d.update(kw)
    return br.BrHparams(**d)


def _desc(br, m, n, geom, src, tau=0):
    return br.BrLayerDesc(m=m, n=n, geom=geom, src=src, grad_dtype=br.BR_F32, tau_max=tau, freq=0, reserved=0, weight=0)


def test_overhead_bytes_match_app_h_table(br):
    """Golden values: tests/golden/memory_table.txt (App. H, Table 2), GiB per matrix in fp32."""
    geoms = {"Bi": br.BR_GEOM_BILATERAL, "Uni": br.BR_GEOM_UNILATERAL}
    srcs = {"2nd": br.BR_SRC_SECOND, "1st": br.BR_SRC_FIRST}
    for line in open(os.path.join(ROOT, "tests", "golden", "memory_table.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        s, g, attn, mlp = line.split()
        for (m, n), printed in (((4096, 4096), float(attn)), ((4096, 14336), float(mlp))):
            _, over = br.br_state_bytes([_desc(br, m, n, geoms[g], srcs[s])], _hp(br))
            assert abs(over / 2 ** 30 - printed) < 0.0051


def test_host_validation(br):
    with pytest.raises(br.BrError) as e:
        br.br_state_bytes([_desc(br, 0, 4, 2, 2)], _hp(br))
    assert e.value.status == br.BR_ERR_SHAPE
    with pytest.raises(br.BrError) as e:
        br.br_state_bytes([_desc(br, 4, 4, 2, 2)], _hp(br, beta1=1.5))
    assert e.value.status == br.BR_ERR_INVALID
    with pytest.raises(br.BrError) as e:
        br.br_state_bytes([_desc(br, 4, 4, 2, 2, tau=-1)], _hp(br))
    assert e.value.status == br.BR_ERR_TAU
    with pytest.raises(br.BrError) as e:
        br.br_state_bytes([_desc(br, 4, 4, 7, 2)], _hp(br))
    assert e.value.status == br.BR_ERR_INVALID
    with pytest.raises(br.BrError) as e:
        br.br_state_bytes([_desc(br, 4, 4, 2, 2)], _hp(br, flags=2))
    assert e.value.status == br.BR_ERR_INVALID
    # the debugging layout adds one 256-byte guard per piece of memory
    plain, _ = br.br_state_bytes([_desc(br, 64, 32, 2, 2, tau=2)], _hp(br))
    guarded, _ = br.br_state_bytes([_desc(br, 64, 32, 2, 2, tau=2)], _hp(br, flags=br.BR_FLAG_DEBUG_CANARY))
    assert guarded > plain and (guarded - plain) % 256 == 0
    assert br.br_strerror(br.BR_ERR_TAU) == "tau out of range"
    assert br.br_destroy(None) == br.BR_OK


def test_create_without_gpu_fails_loudly(br):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(br.BrError) as e:
        br.br_create([br.BrLayerDesc(m=4, n=4, geom=2, src=2, grad_dtype=0, tau_max=0, freq=0, reserved=0, weight=256)],
                     _hp(br), 0, 0, None)
    assert e.value.status == br.BR_ERR_CUDA


def test_ring_total_grows_with_tau(br):
    t0, _ = br.br_state_bytes([_desc(br, 64, 32, 2, 2, tau=0)], _hp(br))
    t4, _ = br.br_state_bytes([_desc(br, 64, 32, 2, 2, tau=4)], _hp(br))
    assert t4 - t0 == 4 * 64 * 32 * 4


def test_stage_aware_helpers_match_the_oracle(br):
    """Host-only helpers of the stage-aware operation (App. I rule, Eq. (effective-delay)) against
    the oracle's rational-arithmetic / numpy statements of the same formulas."""
    import numpy as np
    from oracle import br_oracle as O
    for P in (4, 8, 9, 32, 33):
        for f0 in (1, 10, 14, 50):
            for tau in range(0, P + 3):
                try:
                    want = O.stage_aware_freq(P, tau, f0)
                except ValueError:
                    with pytest.raises(br.BrError) as e:
                        br.br_stage_aware_freq(P, tau, f0)
                    assert e.value.status == br.BR_ERR_INVALID
                    continue
                assert br.br_stage_aware_freq(P, tau, f0) == want, (P, tau, f0)
    rng = np.random.default_rng(0)
    for n in (1, 5, 32):
        c = rng.uniform(0.1, 3.0, n)
        t = rng.integers(0, 32, n)
        assert abs(br.br_effective_delay(c, t) - O.effective_delay(c, t)) < 1e-12
    with pytest.raises(br.BrError):
        br.br_effective_delay([0.0, 0.0], [1, 2])


def test_lr_schedule_helper_matches_the_oracle(br):
    from oracle import br_oracle as O
    for total, frac in ((1000, 0.012), (37, 0.1), (10, 0.0), (5, 1.0)):
        for t in range(total):
            assert abs(br.br_lr_warmup_cosine(t, total, frac, 3e-4, 1e-6) - O.lr_warmup_cosine(t, total, frac, 3e-4, 1e-6)) < 1e-15
    with pytest.raises(br.BrError):
        br.br_lr_warmup_cosine(10, 10, 0.1, 1e-3, 0.0)
