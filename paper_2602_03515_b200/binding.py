"""ctypes binding of include/br.h.  Argument marshalling only: every step of the optimizer path
runs in the CUDA kernels of libbr.so.  torch is used for device memory and streams."""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

BR_OK, BR_WARMUP, BR_WARN_RANK_DEFICIENT = 0, 1, 2
BR_ERR_INVALID, BR_ERR_SHAPE, BR_ERR_DTYPE, BR_ERR_TAU = -1, -2, -3, -4
BR_ERR_OOM, BR_ERR_CUDA, BR_ERR_STATE, BR_ERR_TIMEOUT = -5, -6, -7, -8
BR_GEOM_NONE, BR_GEOM_UNILATERAL, BR_GEOM_BILATERAL = 0, 1, 2
BR_SRC_FIRST, BR_SRC_SECOND = 1, 2
BR_F32, BR_BF16 = 0, 1
BR_GEMM_FP32, BR_GEMM_BF16 = 0, 2
BR_ACCUM_EVERY_STEP, BR_ACCUM_ON_REFRESH = 0, 1
BR_BUF_W, BR_BUF_M, BR_BUF_V2, BR_BUF_U, BR_BUF_V, BR_BUF_L, BR_BUF_R, BR_BUF_RING, BR_BUF_MROT, BR_BUF_CLIP = range(10)


class BrError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"br status {status}: {msg}")
        self.status = status


class BrLayerDesc(C.Structure):
    _fields_ = [("m", C.c_int64), ("n", C.c_int64), ("geom", C.c_int32), ("src", C.c_int32),
                ("grad_dtype", C.c_int32), ("tau_max", C.c_int32), ("freq", C.c_int32),
                ("reserved", C.c_int32), ("weight", C.c_void_p)]


class BrHparams(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("beta_factor", C.c_float), ("freq", C.c_int32),
                ("power_iters", C.c_int32), ("accum", C.c_int32), ("gemm_prec", C.c_int32),
                ("flags", C.c_uint32), ("clip_norm", C.c_float), ("scratch_limit_bytes", C.c_uint64)]


class BrCounters(C.Structure):
    _fields_ = [("calls", C.c_int64), ("t", C.c_int64), ("ring_slot", C.c_int64),
                ("refresh_count", C.c_int64), ("next_refresh_t", C.c_int64), ("basis_flags", C.c_int64)]

    def as_dict(self):
        """The integer state of the method (what the oracle also keeps); `basis_flags` is the library's own
        note on conditioning and is read with br_get_basis_flags."""
        return {k: int(getattr(self, k)) for k, _ in self._fields_ if k != "basis_flags"}


class BrProfileStats(C.Structure):
    _fields_ = [("tc_ms", C.c_double), ("tc_flops", C.c_double), ("tc_launches", C.c_int64),
                ("ema_ms", C.c_double), ("ema_bytes", C.c_double), ("ema_launches", C.c_int64),
                ("refresh_ms", C.c_double), ("refresh_flops", C.c_double), ("refresh_spans", C.c_int64)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


_ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
_FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class BrAllocator(C.Structure):
    _fields_ = [("alloc", _ALLOC_FN), ("free", _FREE_FN), ("ctx", C.c_void_p)]


def library_path() -> str:
    return os.path.join(_HERE, "libbr.so")


def load_library():
    """Load libbr.so (built in-tree by build.py).  Raises if it is missing: no fallback exists."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} not found: build it with `python -m paper_2602_03515_b200.build` "
                          "(there is no CPU or PyTorch fallback for the optimizer path)")
    lib = C.CDLL(path)
    H = C.c_void_p
    sigs = {
        "br_state_bytes": ([C.POINTER(BrLayerDesc), C.c_int, C.POINTER(BrHparams), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)], C.c_int),
        "br_create": ([C.POINTER(H), C.POINTER(BrLayerDesc), C.c_int, C.POINTER(BrHparams), C.c_int, C.c_void_p, C.POINTER(BrAllocator)], C.c_int),
        "br_step": ([H, C.POINTER(C.c_void_p), C.c_int], C.c_int),
        "br_set_lr": ([H, C.c_float], C.c_int),
        "br_refresh_basis": ([H, C.c_int], C.c_int),
        "br_sync_status": ([H], C.c_int),
        "br_get_counters": ([H, C.c_int, C.POINTER(BrCounters)], C.c_int),
        "br_set_counters": ([H, C.c_int, C.POINTER(BrCounters)], C.c_int),
        "br_get_state": ([H, C.c_int, C.c_int, C.c_void_p, C.c_size_t], C.c_int),
        "br_set_state": ([H, C.c_int, C.c_int, C.c_void_p, C.c_size_t], C.c_int),
        "br_get_launch_stats": ([H, C.POINTER(C.c_int64), C.POINTER(C.c_double)], C.c_int),
        "br_profile": ([H, C.c_int], C.c_int),
        "br_get_profile": ([H, C.POINTER(BrProfileStats)], C.c_int),
        "br_stage_aware_freq": ([C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int)], C.c_int),
        "br_effective_delay": ([C.POINTER(C.c_double), C.POINTER(C.c_int), C.c_int, C.POINTER(C.c_double)], C.c_int),
        "br_lr_warmup_cosine": ([C.c_int64, C.c_int64, C.c_double, C.c_double, C.c_double, C.POINTER(C.c_double)], C.c_int),
        "br_destroy": ([H], C.c_int),
        "br_debug_inject": ([H, C.c_int, C.c_int64], C.c_int),
        "br_debug_wait_timeout": ([H, C.c_uint64], C.c_int),
        "br_debug_check_canaries": ([H], C.c_int),
        "br_power_static": ([C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p], C.c_int),
        "br_strerror": ([C.c_int], C.c_char_p),
        "br_last_error": ([H], C.c_char_p),
        "br_gemm_bf16": ([C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.c_int, C.c_int, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_float, C.c_float], C.c_int),
    }
    for name, (argtypes, restype) in sigs.items():
        fn = getattr(lib, name)
        fn.argtypes, fn.restype = argtypes, restype
    _LIB = lib
    return lib


# ---- same-named thin wrappers -------------------------------------------------------------------
def br_strerror(status: int) -> str:
    return load_library().br_strerror(int(status)).decode()


def br_last_error(handle=None) -> str:
    return load_library().br_last_error(handle).decode()


def _check(status: int, handle=None) -> int:
    if status < 0:
        raise BrError(status, f"{br_strerror(status)}: {br_last_error(handle)}")
    return status


def _desc_array(descs: Sequence[BrLayerDesc]):
    arr = (BrLayerDesc * len(descs))()
    for i, d in enumerate(descs):
        arr[i] = d
    return arr


def br_state_bytes(descs: Sequence[BrLayerDesc], hp: BrHparams):
    total, over = C.c_size_t(0), C.c_size_t(0)
    _check(load_library().br_state_bytes(_desc_array(descs), len(descs), C.byref(hp), C.byref(total), C.byref(over)))
    return int(total.value), int(over.value)


def br_create(descs: Sequence[BrLayerDesc], hp: BrHparams, device: int, stream_ptr: int = 0,
              allocator: Optional[BrAllocator] = None):
    h = C.c_void_p()
    st = load_library().br_create(C.byref(h), _desc_array(descs), len(descs), C.byref(hp), int(device),
                                  C.c_void_p(stream_ptr), C.byref(allocator) if allocator is not None else None)
    _check(st, None)
    return h


def br_step(handle, grad_ptrs: Sequence[int], tau: int = -1) -> int:
    arr = (C.c_void_p * len(grad_ptrs))(*[C.c_void_p(p) for p in grad_ptrs])
    return _check(load_library().br_step(handle, arr, int(tau)), handle)


def br_set_lr(handle, lr: float) -> int:
    return _check(load_library().br_set_lr(handle, float(lr)), handle)


def br_refresh_basis(handle, layer: int = -1) -> int:
    return _check(load_library().br_refresh_basis(handle, int(layer)), handle)


def br_sync_status(handle) -> int:
    return _check(load_library().br_sync_status(handle), handle)


def br_get_counters(handle, layer: int) -> dict:
    c = BrCounters()
    _check(load_library().br_get_counters(handle, int(layer), C.byref(c)), handle)
    return c.as_dict()


def br_get_basis_flags(handle, layer: int) -> int:
    c = BrCounters()
    _check(load_library().br_get_counters(handle, int(layer), C.byref(c)), handle)
    return int(c.basis_flags)


def br_set_counters(handle, layer: int, calls: int, t: int, refresh_count: int, basis_flags: int = 0) -> int:
    c = BrCounters(calls=calls, t=t, ring_slot=0, refresh_count=refresh_count, next_refresh_t=0,
                   basis_flags=basis_flags)
    return _check(load_library().br_set_counters(handle, int(layer), C.byref(c)), handle)


def br_get_state(handle, layer: int, which: int, host_ptr: int, nbytes: int) -> int:
    return _check(load_library().br_get_state(handle, int(layer), int(which), C.c_void_p(host_ptr), nbytes), handle)


def br_set_state(handle, layer: int, which: int, host_ptr: int, nbytes: int) -> int:
    return _check(load_library().br_set_state(handle, int(layer), int(which), C.c_void_p(host_ptr), nbytes), handle)


def br_get_launch_stats(handle):
    n, f = C.c_int64(0), C.c_double(0.0)
    _check(load_library().br_get_launch_stats(handle, C.byref(n), C.byref(f)), handle)
    return int(n.value), float(f.value)


def br_profile(handle, enable: bool) -> int:
    return _check(load_library().br_profile(handle, 1 if enable else 0), handle)


def br_get_profile(handle) -> dict:
    st = BrProfileStats()
    _check(load_library().br_get_profile(handle, C.byref(st)), handle)
    return st.as_dict()


def br_stage_aware_freq(P: int, tau: int, f0: int) -> int:
    out = C.c_int(0)
    _check(load_library().br_stage_aware_freq(int(P), int(tau), int(f0), C.byref(out)))
    return int(out.value)


def br_effective_delay(consts, taus) -> float:
    n = len(consts)
    assert n == len(taus)
    cs = (C.c_double * n)(*[float(x) for x in consts])
    ts = (C.c_int * n)(*[int(x) for x in taus])
    out = C.c_double(0.0)
    _check(load_library().br_effective_delay(cs, ts, n, C.byref(out)))
    return float(out.value)


def br_lr_warmup_cosine(step: int, total_steps: int, warmup_fraction: float, base_lr: float, min_lr: float = 0.0) -> float:
    out = C.c_double(0.0)
    _check(load_library().br_lr_warmup_cosine(int(step), int(total_steps), float(warmup_fraction), float(base_lr),
                                              float(min_lr), C.byref(out)))
    return float(out.value)


BR_INJECT_NONE, BR_INJECT_LAUNCH_FAILURE = 0, 1


def br_debug_inject(handle, kind: int, countdown: int = 0) -> int:
    return _check(load_library().br_debug_inject(handle, int(kind), int(countdown)), handle)


BR_FLAG_DEBUG_CANARY = 1


def br_debug_check_canaries(handle) -> int:
    return _check(load_library().br_debug_check_canaries(handle), handle)


def br_debug_wait_timeout(handle, limit_ns: int) -> int:
    return _check(load_library().br_debug_wait_timeout(handle, int(limit_ns)), handle)


def br_destroy(handle) -> int:
    return load_library().br_destroy(handle)


def br_gemm_bf16(stream_ptr, Md, Nd, K, A_ptrs, B_ptrs, a_mn, b_mn, lda, ldb, D_ptr, ldd, alpha=1.0, beta=0.0):
    n = len(A_ptrs)
    A = (C.c_void_p * n)(*[C.c_void_p(p) for p in A_ptrs])
    B = (C.c_void_p * n)(*[C.c_void_p(p) for p in B_ptrs])
    return _check(load_library().br_gemm_bf16(C.c_void_p(stream_ptr), Md, Nd, K, n, A, B, int(a_mn), int(b_mn),
                                              lda, ldb, C.c_void_p(D_ptr), ldd, float(alpha), float(beta)))


def br_power_static(stream_ptr: int, F_ptr: int, Q_ptr: int, k: int, device_flag_ptr: int = 0) -> int:
    """Q <- qr(F Q).Q on the device without allocating; see include/br.h for the limits (k <= 512,
    one shared scratch array per GPU, calls must not overlap on the GPU)."""
    st = load_library().br_power_static(C.c_void_p(stream_ptr), C.c_void_p(F_ptr), C.c_void_p(Q_ptr), int(k),
                                        C.c_void_p(device_flag_ptr) if device_flag_ptr else None)
    if st < 0:
        raise BrError(st, br_strerror(st) + (": order above 512 does not fit the fixed scratch" if st == BR_ERR_SHAPE else ""))
    return st


# ---- convenience object: torch tensors in, pointers out ----------------------------------------------
class BasisRotation:
    """Owns a br_handle.  `weights` are fp32 CUDA tensors updated in place; `specs` give
    (m, n, geom, src, tau_max, freq) per layer (e.g. workloads.LayerSpec)."""

    def __init__(self, specs, weights, *, grad_dtype: str = "bf16", lr=1e-3, beta1=0.9, beta2=0.999,
                 eps=1e-8, weight_decay=0.0, beta_factor=-1.0, freq=10, power_iters=1,
                 accum=BR_ACCUM_EVERY_STEP, gemm_prec=BR_GEMM_BF16, scratch_limit_bytes=0, clip_norm=0.0,
                 flags=0, device=None, stream=None, use_torch_allocator=True):
        import torch
        self._torch = torch
        assert len(specs) == len(weights)
        self.device = torch.device(device if device is not None else weights[0].device)
        if self.device.type != "cuda":
            raise BrError(BR_ERR_CUDA, "the optimizer path runs on a CUDA device only")
        self.weights = list(weights)
        self.specs = list(specs)
        self.grad_dtype = grad_dtype
        gd = BR_BF16 if grad_dtype == "bf16" else BR_F32
        self._descs = []
        for s, w in zip(specs, weights):
            assert w.dtype == torch.float32 and w.is_contiguous() and tuple(w.shape) == (s.m, s.n)
            self._descs.append(BrLayerDesc(m=s.m, n=s.n, geom=s.geom, src=s.src, grad_dtype=gd,
                                           tau_max=s.tau_max, freq=getattr(s, "freq", 0), reserved=0,
                                           weight=w.data_ptr()))
        self.hp = BrHparams(lr=lr, beta1=beta1, beta2=beta2, eps=eps, weight_decay=weight_decay,
                            beta_factor=beta_factor, freq=freq, power_iters=power_iters, accum=accum,
                            gemm_prec=gemm_prec, flags=flags, clip_norm=clip_norm, scratch_limit_bytes=scratch_limit_bytes)
        self._blocks = {}
        self._alloc = None
        if use_torch_allocator:
            dev = self.device

            def _alloc(nbytes, _ctx):
                try:
                    t = torch.empty(int(nbytes), dtype=torch.uint8, device=dev)
                except Exception:
                    return None
                self._blocks[t.data_ptr()] = t
                return t.data_ptr()

            def _free(ptr, _ctx):
                self._blocks.pop(ptr, None)

            self._cb = (_ALLOC_FN(_alloc), _FREE_FN(_free))
            self._alloc = BrAllocator(self._cb[0], self._cb[1], None)
        self.stream = stream
        sp = stream.cuda_stream if stream is not None else torch.cuda.current_stream(self.device).cuda_stream
        idx = self.device.index if self.device.index is not None else torch.cuda.current_device()
        self.handle = br_create(self._descs, self.hp, idx, sp, self._alloc)

    @classmethod
    def from_workload(cls, w, weights, **kw):
        gp = BR_GEMM_FP32 if w.gemm_prec == "f32" else BR_GEMM_BF16
        args = dict(grad_dtype=w.grad_dtype, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                    weight_decay=w.weight_decay, freq=w.freq, gemm_prec=gp)
        args.update(kw)
        return cls(w.layers, weights, **args)

    def state_bytes(self):
        return br_state_bytes(self._descs, self.hp)

    def step(self, grads, tau: int = -1) -> int:
        return br_step(self.handle, [g.data_ptr() for g in grads], tau)

    def set_lr(self, lr: float):
        return br_set_lr(self.handle, lr)

    def refresh_basis(self, layer: int = -1) -> int:
        return br_refresh_basis(self.handle, layer)

    def sync_status(self) -> int:
        return br_sync_status(self.handle)

    def counters(self, layer: int) -> dict:
        return br_get_counters(self.handle, layer)

    def launch_stats(self):
        return br_get_launch_stats(self.handle)

    def profile(self, enable: bool):
        return br_profile(self.handle, enable)

    def get_profile(self) -> dict:
        return br_get_profile(self.handle)

    def _buf_shape(self, layer: int, which: int):
        s = self.specs[layer]
        torch = self._torch
        if which in (BR_BUF_W, BR_BUF_M, BR_BUF_V2, BR_BUF_MROT):
            return (s.m, s.n), torch.float32
        if which in (BR_BUF_U, BR_BUF_L):
            return (s.m, s.m), torch.float32
        if which in (BR_BUF_V, BR_BUF_R):
            return (s.n, s.n), torch.float32
        if which == BR_BUF_CLIP:
            return (max(x.tau_max for x in self.specs) + 1,), torch.float32
        return (s.tau_max, s.m, s.n), (torch.bfloat16 if self.grad_dtype == "bf16" else torch.float32)

    def get_state(self, layer: int, which: int):
        shape, dt = self._buf_shape(layer, which)
        out = self._torch.empty(shape, dtype=dt)
        br_get_state(self.handle, layer, which, out.data_ptr(), out.numel() * out.element_size())
        return out

    def set_state(self, layer: int, which: int, value):
        shape, dt = self._buf_shape(layer, which)
        v = value.detach().to("cpu", dt).contiguous()
        assert tuple(v.shape) == tuple(shape)
        br_set_state(self.handle, layer, which, v.data_ptr(), v.numel() * v.element_size())

    def close(self):
        if getattr(self, "handle", None) is not None:
            br_destroy(self.handle)
            self.handle = None
            self._blocks.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
