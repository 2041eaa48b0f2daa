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
    """Largest entry-wise difference of two bases, column signs removed.  The update is invariant to
    the sign of a basis column, so each column is compared under the sign that fits best; where the
    sign normalisation of the oracle (largest entry positive) is stable this is the same number, and
    it does not jump when two entries of a column nearly tie for the largest."""
    a = np.asarray(q_gpu, dtype=np.float64)
    b = np.asarray(q_ref, dtype=np.float64)
    return float(np.max(np.minimum(np.max(np.abs(a - b), axis=0), np.max(np.abs(a + b), axis=0))))


def factor_accuracy(lay, side, tensor_core):
    """Relative accuracy of the factor the library's refresh starts from, against the oracle's float64
    one.  Tensor-core path, S = 2nd: the product G G^T (G^T G) is accumulated in tensor memory, which
    truncates its fp32 accumulator once per 16-deep slice of the contraction: a relative error of
    0.3 * (c / 16) * 2^-24 for a chain of c contraction indices (measured: 3.6e-6 for an unbroken chain
    of 3072).  The library cuts the contraction into at least ten chunks (at most 256 indices each) that
    it sums in fp32 outside the tensor core, so c = min(256, max(64, K / 10)): 2.5e-7 measured at
    K = 2560.  On top of that comes one fp32 rounding per update of the stored factor.
    S = 1st: the factor is M M^T (M^T M) of the momentum the path keeps in rotated coordinates, built
    from bf16 hi/lo pair products (2^-16 relative).  fp32 path: FFMA accumulation and fp32 storage."""
    if not tensor_core:
        return 2.0 ** -22
    if lay.src == O.SRC_SECOND:
        K = lay.n if side == "U" else lay.m
        chain = min(256.0, max(64.0, K / 10.0))
        return 0.3 * (chain / 16.0) * 2.0 ** -24 + 2.0 ** -24
    return 2.0 ** -15


class _PerturbedLayer(O.OracleLayer):
    """An oracle layer whose factor products carry a relative error: every G G^T (G^T G) entering L (R)
    is multiplied entry-wise by 1 + rel * Z, Z symmetric standard normal, seeded.  Used as a twin of the
    oracle to measure how far the documented accuracy of the library's factor products moves the
    trajectory of the method itself (its conditioning), against which a deviation is then judged."""

    def set_noise(self, rel_left, rel_right, seed):
        self._rel = (rel_left, rel_right)
        self._rng = np.random.default_rng(seed)

    def _noisy(self, P, rel):
        Z = self._rng.standard_normal(P.shape)
        return P * (1.0 + rel * (Z + Z.T) / np.sqrt(2.0))

    def accumulate_factors(self, G, beta):
        if self.L is not None:
            self.L = beta * self.L + (1.0 - beta) * self._noisy(G @ G.T, self._rel[0])
        if self.R is not None:
            self.R = beta * self.R + (1.0 - beta) * self._noisy(G.T @ G, self._rel[1])


class SideBySide:
    """Steps a workload through libbr (GPU) and the oracle (CPU float64) together."""

    def __init__(self, w, *, gemm_prec=None, accum="every_step", power_iters=1, clip_norm=0.0, device="cuda:0",
                 oracle_qr="householder", twin=False, beta_factor=-1.0, **kw):
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
                                    weight_decay=f32(w.weight_decay), clip_norm=f32(clip_norm), qr=oracle_qr,
                                    beta_factor=f32(beta_factor))
        # optional twin of the oracle whose factor products carry the library's documented accuracy
        self.twin = None
        if twin:
            self.twin = O.make_oracle(w, w0, accum=accum, power_iters=power_iters, lr=f32(w.lr), beta1=f32(w.beta1),
                                      beta2=f32(w.beta2), eps=f32(w.eps), weight_decay=f32(w.weight_decay),
                                      clip_norm=f32(clip_norm), qr=oracle_qr)
            for i, lay in enumerate(self.twin.layers):
                lay.__class__ = _PerturbedLayer
                lay.set_noise(factor_accuracy(lay, "U", True), factor_accuracy(lay, "V", True), 1000 + i)
        gp = gemm_prec if gemm_prec is not None else (br.BR_GEMM_FP32 if w.gemm_prec == "f32" else br.BR_GEMM_BF16)
        self.opt = br.BasisRotation.from_workload(
            w, self.weights, gemm_prec=gp, power_iters=power_iters, clip_norm=clip_norm, beta_factor=beta_factor,
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
        self.twin_dev = None
        if self.twin is not None:
            self.twin.step(host, tau)
            self.twin_dev = [None if (a.last_dW is None) else rel_l2(b.last_dW, a.last_dW)
                             for a, b in zip(self.oracle.layers, self.twin.layers)]
        self.torch.cuda.synchronize()
        after = [w.detach().cpu().numpy().astype(np.float64) for w in self.weights]
        dW_g = [a - b for a, b in zip(after, before)]
        # the whole change of the weights (update plus decoupled decay), None on warm-up calls
        dW_o = [None if l.last_dW is None else l.W - b for l, b in zip(self.oracle.layers, before_o)]
        return st_g, st_o, dW_g, dW_o

    def remember_bases(self):
        """Called before a step: the oracle's bases as they are now (a refresh inside the step starts from them)."""
        self._prev = [(None if l.U is None else l.U.copy(), None if l.V is None else l.V.copy()) for l in self.oracle.layers]

    def check_bases(self, layer, tol, v2_tol=None, where="", tensor_core=True):
        """Bases of `layer` (column signs removed, max-abs) and optionally V~ against the oracle's, right
        after a refresh.  The Q factor is unique, but its trailing columns can be fragile: they come out of
        a cancellation against the leading eigen-directions of the factor.  A basis beyond `tol` is
        therefore measured against the oracle's own conditioning of that refresh: it must stay within
        what a perturbation of the oracle's factor of the size of the library's documented factor
        accuracy (`factor_accuracy`) does to the oracle's result -- once per refresh the basis has been
        through, because one power step does not contract a difference inside the nearly degenerate
        noise subspace and the differences of earlier refreshes carry over.  Returns the errors and,
        where that second bound was needed, the bound; a failure reports the smallest pivot
        min_j R_jj / ||a_j|| of the refresh beside the mismatch."""
        br, lay = self.br, self.oracle.layers[layer]
        errs, notes = {}, []
        for idx, (name, which, ref) in enumerate((("U", br.BR_BUF_U, lay.U), ("V", br.BR_BUF_V, lay.V))):
            if ref is None:
                continue
            e = errs[name] = basis_err(self.state(layer, which), ref)
            if e <= tol:
                continue
            Qprev = self._prev[layer][idx]
            if lay.src == O.SRC_SECOND:
                F = lay.L if name == "U" else lay.R
            else:
                F = lay.M @ lay.M.T if name == "U" else lay.M.T @ lay.M
            rel = factor_accuracy(lay, name, tensor_core)
            bound = lay.refresh_count * O.power_sensitivity(F, Qprev, rel=rel, qr=O.QR_IMPLS[self.oracle.hp.qr])
            errs[name + "_conditioning_bound"] = bound
            if e > bound:
                notes.append(f"{name}: {e:.2e} > {tol:g} and > {bound:.2e}, which is how far {lay.refresh_count} relative {rel:.1e} "
                             f"perturbation(s) of the factor move the oracle's own result")
        if v2_tol is not None:
            errs["V2"] = rel_l2(self.state(layer, br.BR_BUF_V2), lay.V2)
            if errs["V2"] > v2_tol:
                notes.append(f"V~: {errs['V2']:.2e} > {v2_tol:g}")
        if notes:
            raise AssertionError(f"{where} layer {layer}: " + "; ".join(notes) + f"; oracle min pivot of this refresh {lay.last_min_pivot}")
        return errs

    def state(self, layer, which):
        return self.opt.get_state(layer, which).float().numpy().astype(np.float64)

    def close(self):
        self.opt.close()
