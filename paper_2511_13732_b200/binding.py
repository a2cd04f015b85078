"""Thin ctypes binding of libpcg.so: argument marshalling only.

Every function mirrors the C entry point of the same name in ``include/pcg.h``.
Tensors are torch CUDA tensors (torch is used for device memory and streams
only); their ``data_ptr()`` is handed to the library unchanged.  There is no
fallback of any kind: if the shared library is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

from . import build as _build

PCG_F32, PCG_BF16, PCG_F16 = 0, 1, 2
FLAG_BAD_DRAFT_TOKEN, FLAG_ZERO_RESIDUAL, FLAG_NONFINITE, FLAG_THINNING_EXHAUSTED = 1, 2, 4, 8
VERIFY_DEFAULT, VERIFY_DENSE, VERIFY_CLUSTER_TERMINAL, VERIFY_BATCHED_TERMINAL = 0, 1, 2, 4
STATUS_NAMES = {0: "PCG_OK", 1: "PCG_ERR_INVALID_ARG", 2: "PCG_ERR_INVALID_GROUPS", 3: "PCG_ERR_UNSUPPORTED",
                4: "PCG_ERR_WORKSPACE", 5: "PCG_ERR_CUDA"}

EXPORTS = [
    "pcg_status_string", "pcg_last_error", "pcg_groups_create", "pcg_groups_destroy", "pcg_groups_info",
    "pcg_groups_set_accept_bias",
    "pcg_group_probs", "pcg_group_probs_workspace_bytes", "pcg_group_probs_ws", "pcg_verify_workspace_bytes", "pcg_verify", "pcg_verify_host_arena_bytes", "pcg_verify_host",
    "pcg_verify_static", "pcg_verify_thinning_workspace_bytes", "pcg_verify_thinning", "pcg_asg_create", "pcg_asg_info", "pcg_asg_csr", "pcg_asg_destroy",
]


class PcgError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class _Csr(ctypes.Structure):
    _fields_ = [("V", ctypes.c_int32), ("M", ctypes.c_int32), ("nnz", ctypes.c_int64),
                ("group_ptr", ctypes.c_void_p), ("group_tok", ctypes.c_void_p), ("tok_degree", ctypes.c_void_p),
                ("weights", ctypes.c_void_p)]


class GroupsInfo(ctypes.Structure):
    _fields_ = [("V", ctypes.c_int32), ("M", ctypes.c_int32), ("nnz", ctypes.c_int64), ("slices", ctypes.c_int32),
                ("slice_len", ctypes.c_int32), ("max_group_size", ctypes.c_int32), ("max_degree", ctypes.c_int32),
                ("device", ctypes.c_int32), ("has_weights", ctypes.c_int32), ("device_bytes", ctypes.c_int64)]


class AsgInfo(ctypes.Structure):
    _fields_ = [("V", ctypes.c_int32), ("M", ctypes.c_int32), ("nnz", ctypes.c_int64),
                ("max_group_size", ctypes.c_int32), ("max_degree", ctypes.c_int32),
                ("similarity_ms", ctypes.c_float), ("total_ms", ctypes.c_float), ("tensor_path", ctypes.c_int32)]


_lib = None


def library_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True):
    """Load libpcg.so (building it first if it is missing or stale and nvcc is present)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if build_if_missing:
        try:
            path = _build.build()
        except (RuntimeError, FileNotFoundError):
            if not os.path.exists(path):
                raise
    lib = ctypes.CDLL(path)
    vp, i32, i64, f32, u32, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_uint32,
                                  ctypes.c_size_t)
    lib.pcg_status_string.argtypes, lib.pcg_status_string.restype = [ctypes.c_int], ctypes.c_char_p
    lib.pcg_last_error.argtypes, lib.pcg_last_error.restype = [], ctypes.c_char_p
    lib.pcg_groups_create.argtypes = [ctypes.POINTER(_Csr), ctypes.c_int, ctypes.POINTER(vp)]
    lib.pcg_groups_create.restype = ctypes.c_int
    lib.pcg_groups_destroy.argtypes, lib.pcg_groups_destroy.restype = [vp], None
    lib.pcg_groups_info.argtypes, lib.pcg_groups_info.restype = [vp, ctypes.POINTER(GroupsInfo)], ctypes.c_int
    lib.pcg_groups_set_accept_bias.argtypes, lib.pcg_groups_set_accept_bias.restype = [vp, f32], ctypes.c_int
    lib.pcg_group_probs.argtypes = [vp, ctypes.c_int, i64, f32, vp, vp, vp]
    lib.pcg_group_probs.restype = ctypes.c_int
    lib.pcg_group_probs_workspace_bytes.argtypes, lib.pcg_group_probs_workspace_bytes.restype = [i32, i32], sz
    lib.pcg_group_probs_ws.argtypes = [vp, ctypes.c_int, i64, f32, vp, vp, vp, sz, vp]
    lib.pcg_group_probs_ws.restype = ctypes.c_int
    lib.pcg_verify_workspace_bytes.argtypes = [i32, i32, i32, i32, ctypes.c_int, u32]
    lib.pcg_verify_workspace_bytes.restype = sz
    lib.pcg_verify.argtypes = [vp, vp, ctypes.c_int, i32, i32, vp, vp, vp, f32, vp, vp, vp, vp, vp, sz, u32, vp, vp]
    lib.pcg_verify.restype = ctypes.c_int
    lib.pcg_verify_host_arena_bytes.argtypes = [i32, i32, i32, i32, ctypes.c_int, u32]
    lib.pcg_verify_host_arena_bytes.restype = sz
    lib.pcg_verify_host.argtypes = [vp, vp, ctypes.c_int, i32, i32, vp, vp, vp, f32, vp, vp, vp, vp, vp, sz, u32, vp]
    lib.pcg_verify_host.restype = ctypes.c_int
    lib.pcg_verify_static.argtypes = [vp, vp, ctypes.c_int, i32, i32, vp, vp, vp, f32, vp, vp, vp, vp, vp]
    lib.pcg_verify_static.restype = ctypes.c_int
    lib.pcg_verify_thinning_workspace_bytes.argtypes = [i32, i32, i32, i32, ctypes.c_int]
    lib.pcg_verify_thinning_workspace_bytes.restype = sz
    lib.pcg_verify_thinning.argtypes = [vp, vp, ctypes.c_int, i32, i32, vp, vp, vp, vp, i32, f32, vp, vp, vp, vp, vp, vp,
                                        sz, vp, vp]
    lib.pcg_verify_thinning.restype = ctypes.c_int
    lib.pcg_asg_create.argtypes = [vp, ctypes.c_int, i32, i32, f32, u32, ctypes.POINTER(vp)]
    lib.pcg_asg_create.restype = ctypes.c_int
    lib.pcg_asg_info.argtypes, lib.pcg_asg_info.restype = [vp, ctypes.POINTER(AsgInfo)], ctypes.c_int
    lib.pcg_asg_csr.argtypes, lib.pcg_asg_csr.restype = [vp, ctypes.POINTER(_Csr)], ctypes.c_int
    lib.pcg_asg_destroy.argtypes, lib.pcg_asg_destroy.restype = [vp], None
    _lib = lib
    return lib


def _check(status: int):
    if status != 0:
        raise PcgError(status, load().pcg_last_error().decode())


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _dev_ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    if stream is None:
        import torch

        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def dtype_code(t) -> int:
    import torch

    if t.dtype == torch.float32:
        return PCG_F32
    if t.dtype == torch.bfloat16 or t.dtype == torch.uint16 or t.dtype == torch.int16:
        return PCG_BF16
    if t.dtype == torch.float16:
        return PCG_F16
    raise TypeError(f"logits must be float32, float16 or bfloat16 (or 16-bit integer bf16 bit patterns), got {t.dtype}")


class Groups:
    """Owner of a ``pcg_groups`` handle built from host numpy arrays (``pcg_groups_create``)."""

    def __init__(self, V: int, group_ptr, group_tok, tok_degree, weights=None, slices_hint: int = 0):
        lib = load()
        self._keep = (np.ascontiguousarray(group_ptr, np.int32), np.ascontiguousarray(group_tok, np.int32),
                      np.ascontiguousarray(tok_degree, np.int32),
                      None if weights is None else np.ascontiguousarray(weights, np.float32))
        gp, gt, dg, w = self._keep
        csr = _Csr(int(V), int(gp.shape[0] - 1), int(gt.shape[0]), _np_ptr(gp), _np_ptr(gt), _np_ptr(dg), _np_ptr(w))
        self.handle = ctypes.c_void_p()
        _check(lib.pcg_groups_create(ctypes.byref(csr), int(slices_hint), ctypes.byref(self.handle)))
        info = GroupsInfo()
        _check(lib.pcg_groups_info(self.handle, ctypes.byref(info)))
        self.info = info
        self.V, self.M = info.V, info.M

    def set_accept_bias(self, bias: float):
        """``pcg_groups_set_accept_bias``: constant added to the acceptance ratio of later ``pcg_verify`` calls."""
        _check(load().pcg_groups_set_accept_bias(self.handle, float(bias)))

    def close(self):
        if getattr(self, "handle", None):
            load().pcg_groups_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def pcg_group_probs_workspace_bytes(V: int, M: int) -> int:
    return int(load().pcg_group_probs_workspace_bytes(int(V), int(M)))


def pcg_group_probs(logits, groups: Groups, temperature: float = 1.0, out=None, stream=None, workspace=None):
    """``pcg_group_probs``: logits [rows, V] (CUDA, float32, bfloat16 or float16) -> float32 [rows, M].

    With ``workspace`` (a uint8 CUDA tensor of at least ``pcg_group_probs_workspace_bytes(V, M)`` bytes) the call goes
    through ``pcg_group_probs_ws`` and touches no scratch of the handle, so calls with separate workspaces may run
    side by side on different streams."""
    import torch

    if logits.dim() != 2 or logits.shape[1] != groups.V or not logits.is_contiguous() or not logits.is_cuda:
        raise ValueError("logits must be a contiguous CUDA tensor [rows, V]")
    rows = logits.shape[0]
    if out is None:
        out = torch.empty((rows, groups.M), dtype=torch.float32, device=logits.device)
    elif tuple(out.shape) != (rows, groups.M) or out.dtype != torch.float32 or not out.is_contiguous() or out.device != logits.device:
        raise ValueError("out must be a contiguous float32 tensor [rows, M] on the logits' device")
    if workspace is None:
        _check(load().pcg_group_probs(_dev_ptr(logits), dtype_code(logits), rows, float(temperature), groups.handle,
                                      _dev_ptr(out), _stream_ptr(stream)))
    else:
        _check(load().pcg_group_probs_ws(_dev_ptr(logits), dtype_code(logits), rows, float(temperature), groups.handle,
                                         _dev_ptr(out), _dev_ptr(workspace), workspace.numel() * workspace.element_size(),
                                         _stream_ptr(stream)))
    return out


def _check_verify_tensors(target_logits, draft_logits, draft_tokens, groups, uniforms, out=None, extra=(), cuda=True):
    """Shapes, types, contiguity and placement of the tensors of a verification call (the library itself only sees
    raw pointers).  ``extra`` lists further (tensor, shape, dtype) triples; ``out`` is the tuple of output tensors
    (accept_len [B], tokens [B, K+1], groups [B, K+1] or None, flags [B] or None, then [B] tensors or None)."""
    import torch

    if target_logits.dim() != 3:
        raise ValueError("target_logits must be [B, K+1, V]")
    B, K1, V = target_logits.shape
    K = K1 - 1
    if V != groups.V:
        raise ValueError(f"the logits have V={V} but the group handle was built for V={groups.V}")
    dev = target_logits.device
    if target_logits.is_cuda != cuda:
        raise ValueError("the tensors of this call must live in %s memory" % ("CUDA" if cuda else "host"))
    checks = [(target_logits, (B, K1, V), target_logits.dtype), (draft_logits, (B, K, V), target_logits.dtype),
              (draft_tokens, (B, K), torch.int32), (uniforms, (B, K + 1, 2), torch.float32)] + list(extra)
    if out is not None:
        shapes = [(B,), (B, K + 1), (B, K + 1), (B,)] + [(B,)] * (len(out) - 4)
        checks += [(t, sh, torch.int32) for t, sh in zip(out, shapes) if t is not None]
        if out[0] is None or out[1] is None:
            raise ValueError("the accept-length and token outputs are required")
    for t, shape, dtype in checks:
        if tuple(t.shape) != tuple(shape) or not t.is_contiguous() or t.device != dev or t.dtype != dtype:
            raise ValueError(f"expected a contiguous {dtype} tensor of shape {tuple(shape)} on {dev}, got "
                             f"{t.dtype} {tuple(t.shape)} on {t.device}")
    return B, K, V


def pcg_verify_workspace_bytes(B: int, K: int, V: int, M: int, dtype: int, mode: int = 0) -> int:
    return int(load().pcg_verify_workspace_bytes(B, K, V, M, dtype, mode))


def pcg_verify(target_logits, draft_logits, draft_tokens, groups: Groups, uniforms, temperature: float = 1.0,
               workspace=None, mode: int = 0, stream=None, want_groups: bool = True, want_flags: bool = True,
               out=None, stage_events=None):
    """``pcg_verify`` on CUDA tensors.  Returns (accept_len [B], tokens [B,K+1], groups or None, flags or None).

    ``workspace`` is a uint8 CUDA tensor of at least ``pcg_verify_workspace_bytes`` bytes (allocated here if
    omitted); ``out`` optionally supplies the four output tensors; ``stage_events`` is a list of three
    ``torch.cuda.Event(enable_timing=True)`` that were recorded at least once (their handles are passed down).
    """
    import torch

    B, K, V = _check_verify_tensors(target_logits, draft_logits, draft_tokens, groups, uniforms, out)
    dev = target_logits.device
    dt = dtype_code(target_logits)
    need = pcg_verify_workspace_bytes(B, K, V, groups.M, dt, mode)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    if out is None:
        accept_len = torch.empty(B, dtype=torch.int32, device=dev)
        tokens = torch.empty((B, K + 1), dtype=torch.int32, device=dev)
        grp = torch.empty((B, K + 1), dtype=torch.int32, device=dev) if want_groups else None
        flags = torch.empty(B, dtype=torch.int32, device=dev) if want_flags else None
    else:
        accept_len, tokens, grp, flags = out
    ev = None
    if stage_events is not None:
        ev = (ctypes.c_void_p * 3)(*[ctypes.c_void_p(e.cuda_event) for e in stage_events])
    _check(load().pcg_verify(_dev_ptr(target_logits), _dev_ptr(draft_logits), dt, B, K, _dev_ptr(draft_tokens),
                             groups.handle, _dev_ptr(uniforms), float(temperature), _dev_ptr(accept_len),
                             _dev_ptr(tokens), _dev_ptr(grp), _dev_ptr(flags), _dev_ptr(workspace),
                             workspace.numel() * workspace.element_size(), mode, _stream_ptr(stream), ev))
    return accept_len, tokens, grp, flags


def pcg_verify_host_arena_bytes(B: int, K: int, V: int, M: int, dtype: int, mode: int = 0) -> int:
    return int(load().pcg_verify_host_arena_bytes(B, K, V, M, dtype, mode))


def pcg_verify_host(target_logits, draft_logits, draft_tokens, groups: Groups, uniforms, temperature: float,
                    arena, out, mode: int = 0, stream=None):
    """``pcg_verify_host``: inputs and the four ``out`` tensors are HOST torch tensors (pinned for speed);
    ``arena`` is a uint8 CUDA tensor of at least ``pcg_verify_host_arena_bytes`` bytes.  Synchronises."""
    B, K, V = _check_verify_tensors(target_logits, draft_logits, draft_tokens, groups, uniforms, out, cuda=False)
    if not arena.is_cuda or arena.element_size() != 1 or not arena.is_contiguous():
        raise ValueError("arena must be a contiguous one-byte-per-element CUDA tensor")
    accept_len, tokens, grp, flags = out
    _check(load().pcg_verify_host(_dev_ptr(target_logits), _dev_ptr(draft_logits), dtype_code(target_logits), B, K,
                                  _dev_ptr(draft_tokens), groups.handle, _dev_ptr(uniforms), float(temperature),
                                  _dev_ptr(accept_len), _dev_ptr(tokens), _dev_ptr(grp), _dev_ptr(flags),
                                  _dev_ptr(arena), arena.numel() * arena.element_size(), mode, _stream_ptr(stream)))
    return out


def pcg_verify_static(target_logits, draft_logits, draft_tokens, groups: Groups, uniforms, temperature: float,
                      out, stream=None):
    """``pcg_verify_static``: verification with the library's built-in scratch.  Every tensor, the four outputs
    in ``out`` included (groups and flags may be None), is supplied by the caller; nothing is allocated here."""
    B, K, V = _check_verify_tensors(target_logits, draft_logits, draft_tokens, groups, uniforms, out)
    accept_len, tokens, grp, flags = out
    _check(load().pcg_verify_static(_dev_ptr(target_logits), _dev_ptr(draft_logits), dtype_code(target_logits), B,
                                    K, _dev_ptr(draft_tokens), groups.handle, _dev_ptr(uniforms),
                                    float(temperature), _dev_ptr(accept_len), _dev_ptr(tokens), _dev_ptr(grp),
                                    _dev_ptr(flags), _stream_ptr(stream)))
    return out


def pcg_verify_thinning_workspace_bytes(B: int, K: int, V: int, M: int, dtype: int) -> int:
    return int(load().pcg_verify_thinning_workspace_bytes(B, K, V, M, dtype))


def pcg_verify_thinning(target_logits, draft_logits, draft_tokens, groups: Groups, uniforms, thin_uniforms,
                        temperature: float = 1.0, workspace=None, stream=None, out=None, stage_events=None):
    """``pcg_verify_thinning`` on CUDA tensors: the terminal group by the paper's thinning sampler.

    ``thin_uniforms`` is [B, n_trials, 3] float32.  Returns (accept_len, tokens, groups, flags, trials); ``out``
    optionally supplies those five tensors (groups, flags and trials may be None).
    """
    import torch

    if thin_uniforms.dim() != 3 or thin_uniforms.shape[2] != 3:
        raise ValueError("thin_uniforms must be [B, n_trials, 3]")
    n_trials = int(thin_uniforms.shape[1])
    B, K, V = _check_verify_tensors(target_logits, draft_logits, draft_tokens, groups, uniforms, out,
                                    extra=[(thin_uniforms, (target_logits.shape[0], n_trials, 3), torch.float32)])
    dev = target_logits.device
    dt = dtype_code(target_logits)
    if workspace is None:
        workspace = torch.empty(pcg_verify_thinning_workspace_bytes(B, K, V, groups.M, dt), dtype=torch.uint8, device=dev)
    if out is None:
        out = (torch.empty(B, dtype=torch.int32, device=dev), torch.empty((B, K + 1), dtype=torch.int32, device=dev),
               torch.empty((B, K + 1), dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev),
               torch.empty(B, dtype=torch.int32, device=dev))
    accept_len, tokens, grp, flags, trials = out
    ev = None
    if stage_events is not None:
        ev = (ctypes.c_void_p * 3)(*[ctypes.c_void_p(e.cuda_event) for e in stage_events])
    _check(load().pcg_verify_thinning(_dev_ptr(target_logits), _dev_ptr(draft_logits), dt, B, K, _dev_ptr(draft_tokens),
                                      groups.handle, _dev_ptr(uniforms), _dev_ptr(thin_uniforms), n_trials,
                                      float(temperature), _dev_ptr(accept_len), _dev_ptr(tokens), _dev_ptr(grp),
                                      _dev_ptr(flags), _dev_ptr(trials), _dev_ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _stream_ptr(stream), ev))
    return out


class Asg:
    """Owner of a ``pcg_asg`` object: groups built on the GPU from an embedding table (``pcg_asg_create``).

    ``emb`` is a contiguous CUDA tensor [V, d], bfloat16 or float32.  ``csr_arrays()`` downloads the result;
    ``groups()`` hands the device-resident CSR straight to ``pcg_groups_create``."""

    def __init__(self, emb, theta: float, mma_sync: bool = False):
        if emb.dim() != 2 or not emb.is_cuda or not emb.is_contiguous():
            raise ValueError("emb must be a contiguous CUDA tensor [V, d]")
        self.handle = ctypes.c_void_p()
        _check(load().pcg_asg_create(_dev_ptr(emb), dtype_code(emb), emb.shape[0], emb.shape[1], float(theta),
                                     1 if mma_sync else 0, ctypes.byref(self.handle)))
        self.info = AsgInfo()
        _check(load().pcg_asg_info(self.handle, ctypes.byref(self.info)))
        self._csr = _Csr()
        _check(load().pcg_asg_csr(self.handle, ctypes.byref(self._csr)))

    def csr_arrays(self):
        """(group_ptr [M+1], group_tok [nnz], tok_degree [V]) as numpy int32 arrays (copied from the device)."""
        import torch

        def fetch(ptr, n):
            if n == 0:
                return np.zeros(0, np.int32)

            class _View:  # zero-copy view of library-owned device memory
                __cuda_array_interface__ = {"shape": (int(n),), "typestr": "<i4", "data": (int(ptr), False), "version": 2}

            return torch.as_tensor(_View(), device="cuda").cpu().numpy().copy()

        i = self.info
        return fetch(self._csr.group_ptr, i.M + 1), fetch(self._csr.group_tok, i.nnz), fetch(self._csr.tok_degree, i.V)

    def groups(self, slices_hint: int = 0) -> "Groups":
        """A verification handle built directly from the device-resident result."""
        g = Groups.__new__(Groups)
        g._keep = (self,)
        g.handle = ctypes.c_void_p()
        _check(load().pcg_groups_create(ctypes.byref(self._csr), int(slices_hint), ctypes.byref(g.handle)))
        g.info = GroupsInfo()
        _check(load().pcg_groups_info(g.handle, ctypes.byref(g.info)))
        g.V, g.M = g.info.V, g.info.M
        return g

    def close(self):
        if getattr(self, "handle", None):
            load().pcg_asg_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
