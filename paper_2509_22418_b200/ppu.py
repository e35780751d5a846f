"""ctypes binding of libppu.so: the same calls as include/ppu.h, argument marshalling only.

PyTorch is used for device memory (the arena, token buffers) and the CUDA stream.  Every step
of the training path runs inside the library's kernels; if the library or a CUDA device is
missing the calls raise - there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libppu.so")

PPU_OK = 0
STATUS = {0: "PPU_OK", -1: "PPU_EINVAL", -2: "PPU_ESHAPE", -3: "PPU_ESUBSET", -4: "PPU_ENOMEM",
          -5: "PPU_ESTATE", -6: "PPU_ECUDA", -7: "PPU_ETIMEOUT", -8: "PPU_ETOKEN"}
SUBSET_FFN_SLICE, SUBSET_FFN_LAYERS, SUBSET_EXPLICIT = 0, 1, 2


class PpuError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{STATUS.get(code, code)}: {msg}")
        self.code = code


class ModelCfg(C.Structure):
    _fields_ = [("n_layer", C.c_int32), ("d_model", C.c_int32), ("n_head", C.c_int32),
                ("d_ff", C.c_int32), ("vocab", C.c_int32), ("max_batch", C.c_int32),
                ("max_seq", C.c_int32), ("ln_eps", C.c_float), ("rope_base", C.c_float),
                ("adam_lr", C.c_float), ("adam_beta1", C.c_float), ("adam_beta2", C.c_float),
                ("adam_eps", C.c_float), ("adam_wd", C.c_float), ("outer_lr", C.c_float),
                ("outer_momentum", C.c_float)]


class SubsetSpec(C.Structure):
    _fields_ = [("n_replicas", C.c_int32), ("mode", C.c_int32), ("n_slices", C.c_int32),
                ("layer_stride", C.c_int32), ("ranges", C.POINTER(C.c_int32)),
                ("train_non_mlp", C.c_int32), ("n_head_slices", C.c_int32),
                ("head_ranges", C.POINTER(C.c_int32))]


class Stats(C.Structure):
    _fields_ = [("param_count", C.c_int64), ("arena_bytes", C.c_int64), ("state_bytes", C.c_int64),
                ("activation_bytes", C.c_int64), ("launches_last_step", C.c_int64),
                ("launches_last_sync", C.c_int64), ("flops_fwd", C.c_double),
                ("flops_dgrad", C.c_double), ("flops_wgrad", C.c_double), ("outer_bytes", C.c_double),
                ("saved_bytes_last_step", C.c_int64)]


CLS_GEMM, CLS_ATTN, CLS_LN, CLS_XENT, CLS_ADAMW, CLS_OUTER, CLS_OTHER, CLS_COUNT = 0, 1, 2, 3, 4, 5, 6, 8
CLS_NAMES = {CLS_GEMM: "gemm", CLS_ATTN: "attention", CLS_LN: "layernorm", CLS_XENT: "cross_entropy",
             CLS_ADAMW: "adamw", CLS_OUTER: "outer", CLS_OTHER: "other"}


class Profile(C.Structure):
    _fields_ = [("ms", C.c_double * CLS_COUNT), ("work", C.c_double * CLS_COUNT),
                ("launches", C.c_int64 * CLS_COUNT), ("dropped", C.c_int64)]

    # the two classes bench.py's roofline is built from
    gemm_ms = property(lambda self: self.ms[CLS_GEMM])
    gemm_flops = property(lambda self: self.work[CLS_GEMM])
    gemm_launches = property(lambda self: self.launches[CLS_GEMM])
    attn_ms = property(lambda self: self.ms[CLS_ATTN])
    attn_flops = property(lambda self: self.work[CLS_ATTN])
    attn_launches = property(lambda self: self.launches[CLS_ATTN])


_lib = None


def lib():
    """Loads libppu.so (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise PpuError(-6, f"{LIB_PATH} is missing: run paper_2509_22418_b200/build.py")
        _lib = C.CDLL(LIB_PATH)
        _lib.ppu_last_error.restype = C.c_char_p
    return _lib


def _check(rc):
    if rc != PPU_OK:
        raise PpuError(rc, lib().ppu_last_error().decode())


def make_cfg(n_layer, d_model, n_head, d_ff, vocab, max_batch, max_seq, ln_eps=1e-5,
             rope_base=1e4, adam_lr=1e-3, adam_beta1=0.9, adam_beta2=0.95, adam_eps=1e-8,
             adam_wd=0.1, outer_lr=0.7, outer_momentum=0.9) -> ModelCfg:
    return ModelCfg(n_layer, d_model, n_head, d_ff, vocab, max_batch, max_seq, ln_eps, rope_base,
                    adam_lr, adam_beta1, adam_beta2, adam_eps, adam_wd, outer_lr, outer_momentum)


def make_spec(n_replicas, mode=SUBSET_FFN_SLICE, n_slices=1, layer_stride=1, ranges=None,
              train_non_mlp=0, n_head_slices=0, head_ranges=None):
    """ranges: int array [K][L][2] for SUBSET_EXPLICIT; head_ranges: optional int array [K][2].
    Returns (spec, keepalive)."""
    keep = []
    ptr = C.POINTER(C.c_int32)()
    hptr = C.POINTER(C.c_int32)()
    if ranges is not None:
        keep.append(np.ascontiguousarray(ranges, dtype=np.int32))
        ptr = keep[-1].ctypes.data_as(C.POINTER(C.c_int32))
    if head_ranges is not None:
        keep.append(np.ascontiguousarray(head_ranges, dtype=np.int32))
        assert keep[-1].shape == (n_replicas, 2)
        hptr = keep[-1].ctypes.data_as(C.POINTER(C.c_int32))
    return SubsetSpec(n_replicas, mode, n_slices, layer_stride, ptr, int(train_non_mlp),
                      int(n_head_slices), hptr), keep


def ppu_query_bytes(cfg: ModelCfg, spec: SubsetSpec) -> int:
    n = C.c_size_t(0)
    _check(lib().ppu_query_bytes(C.byref(cfg), C.byref(spec), C.byref(n)))
    return n.value


def _np_ptr(a, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


class Context:
    """Owns the torch arena and the ppu_ctx handle; methods mirror the C calls."""

    def __init__(self, cfg: ModelCfg, spec: SubsetSpec, keepalive=None, device="cuda:0", stream=None):
        import torch
        if not torch.cuda.is_available():
            raise PpuError(-6, "no CUDA device: this library has no CPU path")
        self.torch = torch
        self.cfg, self.spec, self._keep = cfg, spec, keepalive
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        nbytes = ppu_query_bytes(cfg, spec)
        self.arena = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.arena.data_ptr() + 255) & ~255
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._h = C.c_void_p()
        _check(lib().ppu_create(C.byref(cfg), C.byref(spec), C.c_void_p(base), C.c_size_t(nbytes),
                                C.c_void_p(self.stream.cuda_stream), C.byref(self._h)))
        n = C.c_int64()
        _check(lib().ppu_param_count(self._h, C.byref(n)))
        self.param_count = n.value

    def close(self):
        if self._h:
            lib().ppu_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the four calls of the path ----
    def ppu_local_step(self, replica: int, tokens_dev) -> None:
        assert tokens_dev.is_cuda and tokens_dev.dtype == self.torch.int32 and tokens_dev.is_contiguous()
        b, s = tokens_dev.shape
        _check(lib().ppu_local_step(self._h, replica, C.c_void_p(tokens_dev.data_ptr()), b, s))

    def ppu_local_step_host(self, replica: int, tokens_host: np.ndarray) -> float:
        t = np.ascontiguousarray(tokens_host, dtype=np.int32)
        out = C.c_double()
        _check(lib().ppu_local_step_host(self._h, replica, _np_ptr(t, C.c_int32), t.shape[0],
                                         t.shape[1], C.byref(out)))
        return out.value

    def ppu_outer_sync(self, replicas) -> None:
        r = np.ascontiguousarray(list(replicas), dtype=np.int32)
        _check(lib().ppu_outer_sync(self._h, _np_ptr(r, C.c_int32), len(r)))

    def ppu_outer_sync_group(self, replicas, group: int, n_groups: int) -> None:
        r = np.ascontiguousarray(list(replicas), dtype=np.int32)
        _check(lib().ppu_outer_sync_group(self._h, _np_ptr(r, C.c_int32), len(r), group, n_groups))

    def ppu_loss(self, replica: int) -> float:
        out = C.c_double()
        _check(lib().ppu_loss(self._h, replica, C.byref(out)))
        return out.value

    def ppu_eval_loss(self, replica: int, tokens_dev) -> float:
        b, s = tokens_dev.shape
        out = C.c_double()
        _check(lib().ppu_eval_loss(self._h, replica, C.c_void_p(tokens_dev.data_ptr()), b, s,
                                   C.byref(out)))
        return out.value

    # ---- accessors ----
    def tensors(self):
        n = C.c_int32()
        _check(lib().ppu_tensor_count(self._h, C.byref(n)))
        recs = []
        for i in range(n.value):
            name = C.create_string_buffer(64)
            off, nd = C.c_int64(), C.c_int32()
            shape = (C.c_int64 * 2)()
            _check(lib().ppu_tensor_info(self._h, i, name, 64, C.byref(off), C.byref(nd), shape))
            recs.append((name.value.decode(), off.value, tuple(shape[:nd.value])))
        return recs

    def ppu_set_params(self, theta: np.ndarray, replica: int = -1) -> None:
        t = np.ascontiguousarray(theta, dtype=np.float32)
        _check(lib().ppu_set_params(self._h, replica, _np_ptr(t, C.c_float), C.c_int64(t.size)))

    def ppu_get_params(self, replica: int = -1) -> np.ndarray:
        out = np.empty(self.param_count, dtype=np.float32)
        _check(lib().ppu_get_params(self._h, replica, _np_ptr(out, C.c_float), C.c_int64(out.size)))
        return out

    def ppu_get_working_bf16(self) -> np.ndarray:
        out = np.empty(self.param_count, dtype=np.uint16)
        _check(lib().ppu_get_working_bf16(self._h, _np_ptr(out, C.c_uint16), C.c_int64(out.size)))
        return out

    def ppu_get_outer_momentum(self) -> np.ndarray:
        out = np.empty(self.param_count, dtype=np.float32)
        _check(lib().ppu_get_outer_momentum(self._h, _np_ptr(out, C.c_float), C.c_int64(out.size)))
        return out

    def ppu_set_outer_momentum(self, buf: np.ndarray) -> None:
        t = np.ascontiguousarray(buf, dtype=np.float32)
        _check(lib().ppu_set_outer_momentum(self._h, _np_ptr(t, C.c_float), C.c_int64(t.size)))

    def ppu_subset_count(self, replica: int) -> int:
        n = C.c_int64()
        _check(lib().ppu_subset_count(self._h, replica, C.byref(n)))
        return n.value

    def ppu_subset_index(self, replica: int) -> np.ndarray:
        out = np.empty(self.ppu_subset_count(replica), dtype=np.int64)
        _check(lib().ppu_subset_index(self._h, replica, _np_ptr(out, C.c_int64), C.c_int64(out.size)))
        return out

    def ppu_get_subset_grads(self, replica: int) -> np.ndarray:
        out = np.empty(self.ppu_subset_count(replica), dtype=np.float32)
        _check(lib().ppu_get_subset_grads(self._h, replica, _np_ptr(out, C.c_float),
                                          C.c_int64(out.size)))
        return out

    def ppu_get_subset_state(self, replica: int):
        n = self.ppu_subset_count(replica)
        m, v = np.empty(n, dtype=np.float32), np.empty(n, dtype=np.float32)
        step = C.c_int32()
        _check(lib().ppu_get_subset_state(self._h, replica, _np_ptr(m, C.c_float),
                                          _np_ptr(v, C.c_float), C.byref(step), C.c_int64(n)))
        return m, v, step.value

    def ppu_set_subset_state(self, replica: int, m, v, step: int) -> None:
        n = self.ppu_subset_count(replica)
        mm = None if m is None else np.ascontiguousarray(m, dtype=np.float32)
        vv = None if v is None else np.ascontiguousarray(v, dtype=np.float32)
        _check(lib().ppu_set_subset_state(self._h, replica,
                                          None if mm is None else _np_ptr(mm, C.c_float),
                                          None if vv is None else _np_ptr(vv, C.c_float),
                                          C.c_int32(step), C.c_int64(n)))

    def ppu_replica_values(self, replica: int):
        """The replica's packed trained values as a torch view into the arena (no copy)."""
        ptr, n = C.c_void_p(), C.c_int64()
        _check(lib().ppu_replica_values(self._h, replica, C.byref(ptr), C.byref(n)))
        off = ptr.value - self.arena.data_ptr()
        return self.arena[off:off + 4 * n.value].view(self.torch.float32)

    def ppu_set_backends(self, gemm: int = 0, attention: int = 0) -> None:
        _check(lib().ppu_set_backends(self._h, gemm, attention))

    def ppu_check_guards(self) -> int:
        n = C.c_int64()
        _check(lib().ppu_check_guards(self._h, C.byref(n)))
        return n.value

    def ppu_set_adam_lr(self, lr: float) -> None:
        _check(lib().ppu_set_adam_lr(self._h, C.c_float(lr)))

    def ppu_sync(self) -> None:
        _check(lib().ppu_sync(self._h))

    def ppu_profile_enable(self, enable: bool) -> None:
        _check(lib().ppu_profile_enable(self._h, int(enable)))

    def ppu_profile_read(self) -> Profile:
        p = Profile()
        _check(lib().ppu_profile_read(self._h, C.byref(p)))
        return p

    def ppu_stats(self) -> Stats:
        s = Stats()
        _check(lib().ppu_stats(self._h, C.byref(s)))
        return s


# ---- single-operator entry points (device tensors from torch) ----
def ppu_gemm(A, a_kmajor, B, b_kmajor, M, N, K, out_f32=False, backend=0):
    """A, B: bf16 CUDA tensors, 2-D row-major as stored.  Returns C [M,N]."""
    import torch
    out = torch.empty((M, N), dtype=torch.float32 if out_f32 else torch.bfloat16, device=A.device)
    st = torch.cuda.current_stream(A.device).cuda_stream
    _check(lib().ppu_gemm(C.c_void_p(A.data_ptr()), C.c_int64(A.stride(0)), int(a_kmajor),
                          C.c_void_p(B.data_ptr()), C.c_int64(B.stride(0)), int(b_kmajor),
                          C.c_void_p(out.data_ptr()), C.c_int64(out.stride(0)), int(out_f32),
                          M, N, K, backend, C.c_void_p(st)))
    return out


def ppu_attention_fwd(qkv, batch, seq, n_head, d_head, backend=0):
    import torch
    d = n_head * d_head
    U = torch.empty((batch * seq, d), dtype=torch.bfloat16, device=qkv.device)
    lse = torch.empty((batch, n_head, seq), dtype=torch.float32, device=qkv.device)
    st = torch.cuda.current_stream(qkv.device).cuda_stream
    _check(lib().ppu_attention_fwd(C.c_void_p(qkv.data_ptr()), C.c_void_p(U.data_ptr()),
                                   C.c_void_p(lse.data_ptr()), batch, seq, n_head, d_head, backend,
                                   C.c_void_p(st)))
    return U, lse


def ppu_attention_bwd(qkv, U, lse, dU, batch, seq, n_head, d_head, backend=0):
    import torch
    dqkv = torch.empty_like(qkv)
    scratch = torch.empty((batch * n_head * seq,), dtype=torch.float32, device=qkv.device)
    st = torch.cuda.current_stream(qkv.device).cuda_stream
    _check(lib().ppu_attention_bwd(C.c_void_p(qkv.data_ptr()), C.c_void_p(U.data_ptr()),
                                   C.c_void_p(lse.data_ptr()), C.c_void_p(dU.data_ptr()),
                                   C.c_void_p(dqkv.data_ptr()), C.c_void_p(scratch.data_ptr()),
                                   batch, seq, n_head, d_head, backend, C.c_void_p(st)))
    return dqkv


STATIC_SCRATCH_FLOATS = 1 << 20


def ppu_attention_bwd_static(qkv, U, lse, dU, batch, seq, n_head, d_head, backend=0):
    """Attention backward without caller scratch: for users who cannot allocate device memory
    at the point of the call.  Limited to batch * n_head * seq <= STATIC_SCRATCH_FLOATS."""
    import torch
    dqkv = torch.empty_like(qkv)
    st = torch.cuda.current_stream(qkv.device).cuda_stream
    _check(lib().ppu_attention_bwd_static(C.c_void_p(qkv.data_ptr()), C.c_void_p(U.data_ptr()),
                                          C.c_void_p(lse.data_ptr()), C.c_void_p(dU.data_ptr()),
                                          C.c_void_p(dqkv.data_ptr()), batch, seq, n_head, d_head,
                                          backend, C.c_void_p(st)))
    return dqkv
