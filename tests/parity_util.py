"""Helpers shared by the GPU parity tests: run the C-ABI library and the oracle side by side on
the same seeded inputs (the tests are the only place where both are imported)."""
from __future__ import annotations

import numpy as np

from oracle import br_oracle as O
from workloads import GradientStream, initial_weight


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / (nb if nb > 0 else 1.0))


def basis_err(q_gpu, q_ref):
    return float(np.max(np.abs(O.sign_normalise(np.asarray(q_gpu, dtype=np.float64)) - O.sign_normalise(q_ref))))


class SideBySide:
    """Steps a workload through libbr (GPU) and the oracle (CPU float64) together."""

    def __init__(self, w, *, gemm_prec=None, accum="every_step", power_iters=1, clip_norm=0.0, device="cuda:0",
                 oracle_qr="householder", **kw):
        import torch
        import paper_2602_03515_b200 as br
        self.torch, self.br, self.w = torch, br, w
        self.device = torch.device(device)
        self.streams = [GradientStream(w, i) for i in range(len(w.layers))]
        w0 = [initial_weight(w, i) for i in range(len(w.layers))]
        self.weights = [torch.from_numpy(x.copy()).to(self.device) for x in w0]
        # the C-ABI takes its hyper-parameters as fp32: hand the oracle exactly those values
        f32 = lambda x: float(np.float32(x))
        self.oracle = O.make_oracle(w, w0, accum=accum, power_iters=power_iters, lr=f32(w.lr),
                                    beta1=f32(w.beta1), beta2=f32(w.beta2), eps=f32(w.eps),
                                    weight_decay=f32(w.weight_decay), clip_norm=f32(clip_norm), qr=oracle_qr)
        gp = gemm_prec if gemm_prec is not None else (br.BR_GEMM_FP32 if w.gemm_prec == "f32" else br.BR_GEMM_BF16)
        self.opt = br.BasisRotation.from_workload(
            w, self.weights, gemm_prec=gp, power_iters=power_iters, clip_norm=clip_norm,
            accum=br.BR_ACCUM_ON_REFRESH if accum == "on_refresh" else br.BR_ACCUM_EVERY_STEP, **kw)
        self.call = 0

    def grads_for(self, call):
        torch = self.torch
        host, dev = [], []
        for s in self.streams:
            g32 = s(call)
            host.append(g32)
            if self.w.grad_dtype == "bf16":
                dev.append(torch.from_numpy(s.bits(call).view(np.int16)).view(torch.bfloat16).to(self.device))
            else:
                dev.append(torch.from_numpy(g32).to(self.device))
        return host, dev

    def step(self, tau=-1):
        """Returns (gpu_status, oracle_status, per-layer dW from the GPU, per-layer dW oracle)."""
        self.call += 1
        host, dev = self.grads_for(self.call)
        before = [w.detach().cpu().numpy().astype(np.float64) for w in self.weights]
        before_o = [l.W.copy() for l in self.oracle.layers]
        st_g = self.opt.step(dev, tau)
        st_o = self.oracle.step(host, tau)
        self.torch.cuda.synchronize()
        after = [w.detach().cpu().numpy().astype(np.float64) for w in self.weights]
        dW_g = [a - b for a, b in zip(after, before)]
        # the whole change of the weights (update plus decoupled decay), None on warm-up calls
        dW_o = [None if l.last_dW is None else l.W - b for l, b in zip(self.oracle.layers, before_o)]
        return st_g, st_o, dW_g, dW_o

    def check_bases(self, layer, tol, v2_tol=None, where=""):
        """Bases of `layer` (sign-normalised, max-abs) and optionally V~ against the oracle's.  A failure
        reports the oracle's conditioning of that refresh beside the mismatch: the smallest pivot
        min_j R_jj / ||a_j|| and how far a single fp32 rounding of the factor moves the oracle's own
        result."""
        br, lay = self.br, self.oracle.layers[layer]
        errs = {}
        for name, which, ref in (("U", br.BR_BUF_U, lay.U), ("V", br.BR_BUF_V, lay.V)):
            if ref is None:
                continue
            errs[name] = basis_err(self.state(layer, which), ref)
        if v2_tol is not None:
            errs["V2"] = rel_l2(self.state(layer, br.BR_BUF_V2), lay.V2)
        bad = [k for k, e in errs.items() if e > (v2_tol if k == "V2" else tol)]
        if bad:
            note = f"oracle min pivot {lay.last_min_pivot}"
            if lay.src == O.SRC_SECOND and lay.m * lay.n <= 2048 * 2048:
                F, Q = (lay.L, lay.U) if lay.L is not None else (lay.R, lay.V)
                note += f"; a 2^-24 relative perturbation of the factor moves the oracle's next basis by {O.power_sensitivity(F, Q, qr=O.QR_IMPLS[self.oracle.hp.qr]):.2e}"
            raise AssertionError(f"{where} layer {layer}: {errs} (tolerance {tol}); {note}")
        return errs

    def state(self, layer, which):
        return self.opt.get_state(layer, which).float().numpy().astype(np.float64)

    def close(self):
        self.opt.close()
