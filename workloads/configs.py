"""Layer sets and hyper-parameters of the synthetic workloads C1..C5.

Shapes follow decoder-style transformer blocks (attention and MLP weight
matrices, which are the matrices the method rotates; experimental details in
App. D.2 of the paper); value structure and hyper-parameters follow the
benchmark configurations.  Geometry / source names follow the paper's two
design axes (Sec. 3.2): G in {none, uni, bi}, S in {1st, 2nd}.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional

GEOM_NONE, GEOM_UNI, GEOM_BI = 0, 1, 2
SRC_FIRST, SRC_SECOND = 1, 2


@dataclass(frozen=True)
class LayerSpec:
    name: str
    m: int
    n: int
    geom: int = GEOM_BI
    src: int = SRC_SECOND
    tau_max: int = 0          # ring capacity (slots) for this layer
    freq: int = 0             # 0 -> workload default

    @property
    def numel(self) -> int:
        return self.m * self.n


@dataclass(frozen=True)
class Workload:
    name: str
    layers: List[LayerSpec]
    grad_dtype: str           # "f32" | "bf16"
    grad_kind: str            # "iid_normal" | "lowrank_noise" | "student_t"
    grad_scale: float         # iid: sigma; lowrank: noise sigma; student_t: scale
    grad_rank: int = 0        # lowrank_noise only
    tau: int = 0
    freq: int = 10
    calls: int = 0
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.0
    gemm_prec: str = "bf16"   # "f32" | "bf16"
    seed: int = 0
    notes: str = ""

    @property
    def n_params(self) -> int:
        return sum(l.numel for l in self.layers)


def _block(d: int, ffn: int, fused_qkv: bool, gated: bool, geom: int, src: int,
           tau: int, prefix: str = "") -> List[LayerSpec]:
    mk = lambda nm, m, n: LayerSpec(prefix + nm, m, n, geom, src, tau)
    out: List[LayerSpec] = []
    if fused_qkv:
        out += [mk("Wqkv", d, 3 * d), mk("Wo", d, d)]
    else:
        out += [mk("Wq", d, d), mk("Wk", d, d), mk("Wv", d, d), mk("Wo", d, d)]
    if gated:
        out += [mk("Wgate", d, ffn), mk("Wup", d, ffn), mk("Wdown", ffn, d)]
    else:
        out += [mk("W1", d, ffn), mk("W2", ffn, d)]
    return out


def _decoder(n_layers: int, d: int, ffn: int, vocab: int, tau: int) -> List[LayerSpec]:
    layers: List[LayerSpec] = []
    for i in range(n_layers):
        layers += _block(d, ffn, False, True, GEOM_BI, SRC_SECOND, tau, prefix=f"L{i}.")
    # Embedding handled unilaterally (rotation on the smaller, d_model side).
    layers.append(LayerSpec("embed", vocab, d, GEOM_UNI, SRC_SECOND, tau))
    return layers


WORKLOAD_NAMES = ("c1", "c2", "c3", "c4", "c5")


def get_workload(name: str, n_layers: Optional[int] = None, tau: Optional[int] = None) -> Workload:
    """Return workload `name`; `n_layers`/`tau` override depth / delay (c4, c5)."""
    name = name.lower()
    if name == "c1":
        w = Workload("c1", [LayerSpec("W", 64, 32, GEOM_BI, SRC_SECOND, 2)], "f32", "iid_normal",
                     0.01, tau=2, freq=5, calls=20, gemm_prec="f32", seed=0)
    elif name == "c2":
        w = Workload("c2", _block(1024, 4096, True, False, GEOM_BI, SRC_SECOND, 4), "bf16",
                     "lowrank_noise", 0.1, 16, tau=4, freq=10, calls=100, seed=0)
    elif name == "c3":
        w = Workload("c3", _block(1024, 4096, True, False, GEOM_UNI, SRC_FIRST, 8), "bf16",
                     "lowrank_noise", 0.1, 16, tau=8, freq=10, calls=100, seed=0)
    elif name == "c4":
        t = 16 if tau is None else tau
        w = Workload("c4", _decoder(n_layers or 24, 2048, 5632, 32000, t), "bf16", "student_t",
                     1e-3, tau=t, freq=20, calls=50, seed=0)
    elif name == "c5":
        t = 32 if tau is None else tau
        w = Workload("c5", _decoder(n_layers or 32, 2560, 6912, 32000, t), "bf16",
                     "lowrank_noise", 0.05, 32, tau=t, freq=50, calls=20, seed=0)
    else:
        raise KeyError(f"unknown workload {name!r}; choose from {WORKLOAD_NAMES}")
    if tau is not None and name in ("c1", "c2", "c3"):
        w = replace(w, tau=tau, layers=[replace(l, tau_max=tau) for l in w.layers])
    return w


def scaled(w: Workload, div: int, min_dim: int = 8) -> Workload:
    """Same structure with every dimension divided by `div` (parity-sized cases)."""
    ls = [replace(l, m=max(min_dim, l.m // div), n=max(min_dim, l.n // div)) for l in w.layers]
    return replace(w, layers=ls, name=f"{w.name}/div{div}")
