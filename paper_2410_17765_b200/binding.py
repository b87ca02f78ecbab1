"""ctypes binding of libcpmtp.so: argument marshalling only.

Every step of the computation runs in the library's CUDA kernels; torch is used
for device memory and the current stream.  There is no fallback: if the shared
library is missing or fails to load, importing this module's functions raises.
"""
from __future__ import annotations

import contextlib
import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

from .build import DEBUG_LIB_PATH, LIB_PATH

OP_FORWARD, OP_BACKWARD, OP_SCORE, OP_SAMPLE, OP_FORWARD_FULL, OP_BACKWARD_FULL = 0, 1, 2, 3, 4, 5
OP_DISTILL_FORWARD, OP_DISTILL_BACKWARD = 6, 7
FLAG_AUX = 1
FLAG_PER_TOKEN = 2
FLAG_RECOMPUTE_Z = 4
FLAG_ACCUM_GRADS = 8

EXPORTS = [
    "cpmtp_version", "cpmtp_status_string", "cpmtp_workspace_bytes", "cpmtp_forward", "cpmtp_backward",
    "cpmtp_score_draft", "cpmtp_host_staging_bytes", "cpmtp_forward_host", "cpmtp_profile_begin",
    "cpmtp_profile_end", "cpmtp_score_draft_static", "cpmtp_sample_draft",
    "cpmtp_forward_full", "cpmtp_backward_full", "cpmtp_verify_draft",
    "cpmtp_distill_forward", "cpmtp_distill_backward", "cpmtp_reload_knobs", "cpmtp_debug_status",
]

STATIC_SCRATCH_BYTES = 4 << 20

STAGES = ["gate", "proj", "lse", "mixture", "finalize", "coeff", "logit_grad", "dz", "de", "de_convert",
          "dw_head", "dh", "dw_g", "draft_step", "teacher_lse", "kl"]


class CShape(ctypes.Structure):
    _fields_ = [("N", ctypes.c_int32), ("d", ctypes.c_int32), ("V", ctypes.c_int32), ("n", ctypes.c_int32),
                ("r", ctypes.c_int32), ("flags", ctypes.c_uint32), ("aux_coef", ctypes.c_float)]


class CSaved(ctypes.Structure):
    _fields_ = [("lse", ctypes.c_void_p), ("tgt", ctypes.c_void_p), ("logw", ctypes.c_void_p),
                ("q", ctypes.c_void_p), ("wbar", ctypes.c_void_p), ("z", ctypes.c_void_p)]


class CDistillSaved(ctypes.Structure):
    _fields_ = [("lse_t", ctypes.c_void_p), ("logpi", ctypes.c_void_p), ("pm", ctypes.c_void_p),
                ("kl", ctypes.c_void_p)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libcpmtp.so (built in-tree by build.py); raise if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    # CPMTP_LIBRARY=debug selects the checked build (index checks in every epilogue), made by
    # `python -m paper_2410_17765_b200.build --debug`; any other value is taken as a path
    choice = os.environ.get("CPMTP_LIBRARY", "")
    path = LIB_PATH if not choice else DEBUG_LIB_PATH if choice == "debug" else choice
    if not os.path.exists(path):
        raise RuntimeError(f"{path} not found: build it with `python -m paper_2410_17765_b200.build`")
    lib = ctypes.CDLL(path)
    vp, sz, i32p, fp = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p
    shp = ctypes.POINTER(CShape)
    svp = ctypes.POINTER(CSaved)
    lib.cpmtp_version.restype = ctypes.c_int
    lib.cpmtp_status_string.restype = ctypes.c_char_p
    lib.cpmtp_status_string.argtypes = [ctypes.c_int]
    lib.cpmtp_workspace_bytes.restype = sz
    lib.cpmtp_workspace_bytes.argtypes = [shp, ctypes.c_int]
    lib.cpmtp_host_staging_bytes.restype = sz
    lib.cpmtp_host_staging_bytes.argtypes = [shp]
    lib.cpmtp_forward.restype = ctypes.c_int
    lib.cpmtp_forward.argtypes = [shp, vp, vp, vp, vp, i32p, fp, fp, svp, i32p, vp, sz, i32p, vp]
    lib.cpmtp_backward.restype = ctypes.c_int
    lib.cpmtp_backward.argtypes = [shp, vp, vp, vp, vp, i32p, svp, fp, vp, vp, vp, vp, vp, sz, i32p, vp]
    lib.cpmtp_score_draft.restype = ctypes.c_int
    lib.cpmtp_score_draft.argtypes = [shp, vp, vp, vp, vp, i32p, fp, fp, vp, sz, i32p, vp]
    lib.cpmtp_forward_host.restype = ctypes.c_int
    lib.cpmtp_forward_host.argtypes = [shp, vp, vp, vp, vp, i32p, fp, fp, svp, vp, sz, i32p, vp]
    lib.cpmtp_sample_draft.restype = ctypes.c_int
    lib.cpmtp_sample_draft.argtypes = [shp, vp, vp, vp, vp, fp, ctypes.c_float, ctypes.c_int32, i32p, i32p, fp, i32p,
                                       fp, vp, sz, i32p, vp]
    lib.cpmtp_forward_full.restype = ctypes.c_int
    lib.cpmtp_forward_full.argtypes = [shp, vp, vp, vp, i32p, fp, fp, fp, svp, i32p, vp, sz, i32p, vp]
    lib.cpmtp_backward_full.restype = ctypes.c_int
    lib.cpmtp_backward_full.argtypes = [shp, vp, vp, vp, i32p, svp, fp, vp, vp, vp, vp, sz, i32p, vp]
    lib.cpmtp_verify_draft.restype = ctypes.c_int
    lib.cpmtp_verify_draft.argtypes = [ctypes.c_int32, ctypes.c_int32, i32p, i32p, fp, fp, fp, i32p, vp]
    lib.cpmtp_score_draft_static.restype = ctypes.c_int
    lib.cpmtp_score_draft_static.argtypes = [shp, vp, vp, vp, vp, i32p, fp, fp, i32p, vp]
    dsp = ctypes.POINTER(CDistillSaved)
    lib.cpmtp_distill_forward.restype = ctypes.c_int
    lib.cpmtp_distill_forward.argtypes = [shp, vp, vp, vp, vp, i32p, vp, ctypes.c_float, ctypes.c_float, fp, fp, fp,
                                          svp, dsp, vp, sz, i32p, vp]
    lib.cpmtp_distill_backward.restype = ctypes.c_int
    lib.cpmtp_distill_backward.argtypes = [shp, vp, vp, vp, vp, i32p, vp, svp, dsp, ctypes.c_float, ctypes.c_float,
                                           fp, fp, vp, vp, vp, vp, vp, sz, i32p, vp]
    lib.cpmtp_reload_knobs.restype = ctypes.c_int
    lib.cpmtp_debug_status.restype = ctypes.c_int
    lib.cpmtp_profile_begin.restype = ctypes.c_int
    lib.cpmtp_profile_end.restype = ctypes.c_int
    lib.cpmtp_profile_end.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32), ctypes.c_int]
    _lib = lib
    return lib


def debug_status() -> int:
    """cpmtp_debug_status: -1 for the release library; for the checked build 0 while every index check has
    passed and 3 once one has failed (synchronizes the device)."""
    return int(load_library().cpmtp_debug_status())


def reload_knobs() -> None:
    """cpmtp_reload_knobs: have the library read its CPMTP_* environment knobs again."""
    _check(load_library().cpmtp_reload_knobs())


@contextlib.contextmanager
def knobs(**values):
    """Set CPMTP_* environment knobs (name=value; None leaves a knob alone) for the calls made inside the
    block, then restore the environment; the library re-reads its knobs on entry and on exit."""
    values = {k: v for k, v in values.items() if v is not None}
    old = {k: os.environ.get(k) for k in values}
    try:
        for k, v in values.items():
            os.environ[k] = str(v)
        reload_knobs()
        yield
    finally:
        for k, v in old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v
        reload_knobs()


def profile_begin() -> None:
    _check(load_library().cpmtp_profile_begin())


def profile_end() -> dict:
    """Stop per-stage timing; returns {stage: (total_ms, launches)} for stages that ran."""
    n = len(STAGES)
    ms = (ctypes.c_float * n)()
    cnt = (ctypes.c_int32 * n)()
    total = load_library().cpmtp_profile_end(ms, cnt, n)
    if total < 0:
        _check(total)
    return {STAGES[i]: (float(ms[i]), int(cnt[i])) for i in range(n) if cnt[i] > 0}


class CpmtpError(RuntimeError):
    pass


def _check(rc: int) -> None:
    if rc != 0:
        raise CpmtpError(f"cpmtp error {rc}: {load_library().cpmtp_status_string(rc).decode()}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_shape(N, d, V, n, r, aux_coef: Optional[float] = None) -> CShape:
    flags = FLAG_AUX if aux_coef is not None else 0
    return CShape(N, d, V, n, r, flags, float(aux_coef or 0.0))


def workspace_bytes(shape: CShape, op: int) -> int:
    return int(load_library().cpmtp_workspace_bytes(ctypes.byref(shape), op))


def host_staging_bytes(shape: CShape) -> int:
    return int(load_library().cpmtp_host_staging_bytes(ctypes.byref(shape)))


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


@dataclass
class Saved:
    """Forward results kept for cpmtp_backward (device tensors)."""
    lse: torch.Tensor
    tgt: torch.Tensor
    logw: torch.Tensor
    q: torch.Tensor
    wbar: torch.Tensor
    z: torch.Tensor

    @staticmethod
    def alloc_full(shape: CShape, device="cuda") -> "Saved":
        """Saved state for the full-head entry points (no projected hidden states)."""
        K = shape.n * shape.r
        f = dict(dtype=torch.float32, device=device)
        return Saved(lse=torch.empty((shape.N, K), **f), tgt=torch.empty((shape.N, K), **f),
                     logw=torch.empty((shape.N, shape.r), **f), q=torch.empty((shape.N, shape.r), **f),
                     wbar=torch.empty((32,), **f), z=torch.empty(8, dtype=torch.bfloat16, device=device))

    @staticmethod
    def alloc(shape: CShape, device="cuda") -> "Saved":
        K = shape.n * shape.r
        f = dict(dtype=torch.float32, device=device)
        return Saved(lse=torch.empty((shape.N, K), **f), tgt=torch.empty((shape.N, K), **f),
                     logw=torch.empty((shape.N, shape.r), **f), q=torch.empty((shape.N, shape.r), **f),
                     wbar=torch.empty((32,), **f),
                     z=torch.empty((shape.N, K, shape.d), dtype=torch.bfloat16, device=device))

    def c_struct(self) -> CSaved:
        return CSaved(self.lse.data_ptr(), self.tgt.data_ptr(), self.logw.data_ptr(), self.q.data_ptr(),
                      self.wbar.data_ptr(), self.z.data_ptr() if self.z is not None else None)


def _shape_of(h, W_head, E, W_g, x, aux_coef) -> CShape:
    N, d = h.shape
    V = E.shape[0]
    n = x.shape[1]
    r = W_g.shape[0]
    assert W_head.shape == (n * r, d, d) and E.shape[1] == d and W_g.shape[1] == d and x.shape[0] == N
    for t in (h, W_head, E, W_g):
        assert t.dtype == torch.bfloat16 and t.is_contiguous()
    assert x.dtype == torch.int32 and x.is_contiguous()
    return make_shape(N, d, V, n, r, aux_coef)


def forward(h, W_head, E, W_g, x, *, aux_coef: Optional[float] = None, saved: Optional[Saved] = None,
            want_loss: bool = True, want_counts: bool = False, workspace: Optional[torch.Tensor] = None,
            dev_status: Optional[torch.Tensor] = None, out: Optional[dict] = None,
            recompute_z: bool = False) -> dict:
    """cpmtp_forward on device tensors; returns {"logp", "loss", "counts"} (device tensors).
    recompute_z: do not keep z in `saved` (CPMTP_FLAG_RECOMPUTE_Z; pass the same to backward)."""
    lib = load_library()
    shape = _shape_of(h, W_head, E, W_g, x, aux_coef)
    if recompute_z:
        shape.flags |= FLAG_RECOMPUTE_Z
    dev = h.device
    if workspace is None:
        workspace = alloc_workspace(workspace_bytes(shape, OP_FORWARD), dev)
    res = out if out is not None else {}
    if "logp" not in res:
        res["logp"] = torch.empty(shape.N, dtype=torch.float32, device=dev)
    if want_loss and "loss" not in res:
        res["loss"] = torch.empty(1, dtype=torch.float32, device=dev)
    if want_counts and "counts" not in res:
        res["counts"] = torch.empty(shape.r, dtype=torch.int32, device=dev)
    cs = saved.c_struct() if saved is not None else None
    rc = lib.cpmtp_forward(ctypes.byref(shape), _ptr(h), _ptr(W_head), _ptr(E), _ptr(W_g), _ptr(x),
                           _ptr(res["logp"]), _ptr(res.get("loss")) if want_loss else None,
                           ctypes.byref(cs) if cs is not None else None,
                           _ptr(res.get("counts")) if want_counts else None, _ptr(workspace),
                           workspace.numel(), _ptr(dev_status), _stream())
    _check(rc)
    return res


def backward(h, W_head, E, W_g, x, saved: Saved, *, aux_coef: Optional[float] = None,
             dloss_dlogp: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
             dev_status: Optional[torch.Tensor] = None, out: Optional[dict] = None,
             skip: tuple = (), dloss_dprefix: Optional[torch.Tensor] = None,
             recompute_z: bool = False, accumulate: bool = False) -> dict:
    """cpmtp_backward on device tensors; returns {"dh", "dW_head", "dE", "dW_g"} (bf16 device tensors).
    Names listed in `skip` are not computed (passed as NULL).  dloss_dprefix [N, n] fp32 selects the
    per-token objective sum_i sum_s dloss_dprefix[i, s] * log P(x[i, 0..s]) (CPMTP_FLAG_PER_TOKEN).
    accumulate: add to the tensors given in `out` instead of overwriting them (CPMTP_FLAG_ACCUM_GRADS)."""
    lib = load_library()
    shape = _shape_of(h, W_head, E, W_g, x, aux_coef)
    if recompute_z:
        shape.flags |= FLAG_RECOMPUTE_Z
    if accumulate:
        assert out is not None, "accumulation needs the tensors to add to"
        shape.flags |= FLAG_ACCUM_GRADS
    if dloss_dprefix is not None:
        assert dloss_dlogp is None and dloss_dprefix.shape == (shape.N, shape.n) and dloss_dprefix.dtype == torch.float32
        shape.flags |= FLAG_PER_TOKEN
        dloss_dlogp = dloss_dprefix.contiguous()
    if workspace is None:
        workspace = alloc_workspace(workspace_bytes(shape, OP_BACKWARD), h.device)
    res = out if out is not None else {}
    for name, ref in (("dh", h), ("dW_head", W_head), ("dE", E), ("dW_g", W_g)):
        if name not in res and name not in skip:
            res[name] = torch.empty_like(ref)
    cs = saved.c_struct()
    rc = lib.cpmtp_backward(ctypes.byref(shape), _ptr(h), _ptr(W_head), _ptr(E), _ptr(W_g), _ptr(x),
                            ctypes.byref(cs), _ptr(dloss_dlogp), _ptr(res.get("dh")), _ptr(res.get("dW_head")),
                            _ptr(res.get("dE")), _ptr(res.get("dW_g")), _ptr(workspace), workspace.numel(),
                            _ptr(dev_status), _stream())
    _check(rc)
    return res


def score_draft(h, W_head, E, W_g, draft, *, want_prefix: bool = True,
                workspace: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                out: Optional[dict] = None) -> dict:
    """cpmtp_score_draft; returns {"logp_joint", "logp_prefix"} (device tensors)."""
    lib = load_library()
    shape = _shape_of(h, W_head, E, W_g, draft, None)
    if workspace is None:
        workspace = alloc_workspace(workspace_bytes(shape, OP_SCORE), h.device)
    res = out if out is not None else {}
    if "logp_joint" not in res:
        res["logp_joint"] = torch.empty(shape.N, dtype=torch.float32, device=h.device)
    if want_prefix and "logp_prefix" not in res:
        res["logp_prefix"] = torch.empty((shape.N, shape.n), dtype=torch.float32, device=h.device)
    rc = lib.cpmtp_score_draft(ctypes.byref(shape), _ptr(h), _ptr(W_head), _ptr(E), _ptr(W_g), _ptr(draft),
                               _ptr(res["logp_joint"]), _ptr(res.get("logp_prefix")) if want_prefix else None,
                               _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream())
    _check(rc)
    return res


def sample_draft(h, W_head, E, W_g, n: int, *, uniform: Optional[torch.Tensor] = None, temperature: float = 1.0,
                 topk: int = 1, forced: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                 dev_status: Optional[torch.Tensor] = None, out: Optional[dict] = None) -> dict:
    """cpmtp_sample_draft; returns {"draft", "logp_joint", "topk_tokens", "topk_logp"} (device tensors).
    uniform: [N, n, V] fp32 strictly inside (0, 1) for Gumbel-max sampling, or None for the greedy draft.
    forced: [N, n] int32, entries >= 0 fix the token of that step (-1: left to the sampler), or None."""
    lib = load_library()
    N, d = h.shape
    V, r = E.shape[0], W_g.shape[0]
    assert W_head.shape == (n * r, d, d)
    for t in (h, W_head, E, W_g):
        assert t.dtype == torch.bfloat16 and t.is_contiguous()
    if uniform is not None:
        assert uniform.shape == (N, n, V) and uniform.dtype == torch.float32 and uniform.is_contiguous()
    if forced is not None:
        assert forced.shape == (N, n) and forced.dtype == torch.int32 and forced.is_contiguous()
    shape = make_shape(N, d, V, n, r)
    if workspace is None:
        workspace = alloc_workspace(workspace_bytes(shape, OP_SAMPLE), h.device)
    res = out if out is not None else {}
    dev = h.device
    res.setdefault("draft", torch.empty((N, n), dtype=torch.int32, device=dev))
    res.setdefault("logp_joint", torch.empty(N, dtype=torch.float32, device=dev))
    res.setdefault("topk_tokens", torch.empty((N, n, topk), dtype=torch.int32, device=dev))
    res.setdefault("topk_logp", torch.empty((N, n, topk), dtype=torch.float32, device=dev))
    rc = lib.cpmtp_sample_draft(ctypes.byref(shape), _ptr(h), _ptr(W_head), _ptr(E), _ptr(W_g), _ptr(uniform),
                                ctypes.c_float(temperature), topk, _ptr(forced), _ptr(res["draft"]),
                                _ptr(res["logp_joint"]),
                                _ptr(res["topk_tokens"]), _ptr(res["topk_logp"]), _ptr(workspace), workspace.numel(),
                                _ptr(dev_status), _stream())
    _check(rc)
    return res


def _shape_full(h, W_full, W_g, x, aux_coef) -> CShape:
    N, d = h.shape
    K, V, d2 = W_full.shape
    n, r = x.shape[1], W_g.shape[0]
    assert K == n * r and d2 == d and W_g.shape[1] == d and x.shape[0] == N
    for t in (h, W_full, W_g):
        assert t.dtype == torch.bfloat16 and t.is_contiguous()
    assert x.dtype == torch.int32 and x.is_contiguous()
    return make_shape(N, d, V, n, r, aux_coef)


def forward_full(h, W_full, W_g, x, *, aux_coef: Optional[float] = None, saved: Optional[Saved] = None,
                 want_prefix: bool = False, workspace: Optional[torch.Tensor] = None,
                 dev_status: Optional[torch.Tensor] = None, out: Optional[dict] = None) -> dict:
    """cpmtp_forward_full (W_full [n*r, V, d]); returns {"logp", "loss", "counts"[, "logp_prefix"]}."""
    lib = load_library()
    shape = _shape_full(h, W_full, W_g, x, aux_coef)
    dev = h.device
    if workspace is None:
        workspace = alloc_workspace(workspace_bytes(shape, OP_FORWARD_FULL), dev)
    res = out if out is not None else {}
    res.setdefault("logp", torch.empty(shape.N, dtype=torch.float32, device=dev))
    res.setdefault("loss", torch.empty(1, dtype=torch.float32, device=dev))
    res.setdefault("counts", torch.empty(shape.r, dtype=torch.int32, device=dev))
    if want_prefix:
        res.setdefault("logp_prefix", torch.empty((shape.N, shape.n), dtype=torch.float32, device=dev))
    cs = saved.c_struct() if saved is not None else None
    rc = lib.cpmtp_forward_full(ctypes.byref(shape), _ptr(h), _ptr(W_full), _ptr(W_g), _ptr(x), _ptr(res["logp"]),
                                _ptr(res["loss"]), _ptr(res.get("logp_prefix")) if want_prefix else None,
                                ctypes.byref(cs) if cs is not None else None, _ptr(res["counts"]), _ptr(workspace),
                                workspace.numel(), _ptr(dev_status), _stream())
    _check(rc)
    return res


def backward_full(h, W_full, W_g, x, saved: Saved, *, aux_coef: Optional[float] = None,
                  dloss_dlogp: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                  dev_status: Optional[torch.Tensor] = None, out: Optional[dict] = None,
                  dloss_dprefix: Optional[torch.Tensor] = None, accumulate: bool = False) -> dict:
    """cpmtp_backward_full; returns {"dh", "dW_full", "dW_g"} (bf16 device tensors).
    dloss_dprefix and accumulate as for backward()."""
    lib = load_library()
    shape = _shape_full(h, W_full, W_g, x, aux_coef)
    if accumulate:
        assert out is not None, "accumulation needs the tensors to add to"
        shape.flags |= FLAG_ACCUM_GRADS
    if dloss_dprefix is not None:
        assert dloss_dlogp is None and dloss_dprefix.shape == (shape.N, shape.n) and dloss_dprefix.dtype == torch.float32
        shape.flags |= FLAG_PER_TOKEN
        dloss_dlogp = dloss_dprefix.contiguous()
    if workspace is None:
        workspace = alloc_workspace(workspace_bytes(shape, OP_BACKWARD_FULL), h.device)
    res = out if out is not None else {}
    for name, ref in (("dh", h), ("dW_full", W_full), ("dW_g", W_g)):
        if name not in res:
            res[name] = torch.empty_like(ref)
    cs = saved.c_struct()
    rc = lib.cpmtp_backward_full(ctypes.byref(shape), _ptr(h), _ptr(W_full), _ptr(W_g), _ptr(x), ctypes.byref(cs),
                                 _ptr(dloss_dlogp), _ptr(res["dh"]), _ptr(res["dW_full"]), _ptr(res["dW_g"]),
                                 _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream())
    _check(rc)
    return res


def verify_draft(draft: Optional[torch.Tensor] = None, base_tokens: Optional[torch.Tensor] = None, *,
                 logp_prefix: Optional[torch.Tensor] = None, logp_base: Optional[torch.Tensor] = None,
                 uniform: Optional[torch.Tensor] = None) -> torch.Tensor:
    """cpmtp_verify_draft: accepted draft length per position (int32 device tensor).
    Greedy: pass draft and base_tokens [N, n]; probabilistic: pass logp_prefix, logp_base, uniform [N, n]."""
    ref = base_tokens if base_tokens is not None else logp_prefix
    N, n = ref.shape
    accepted = torch.empty(N, dtype=torch.int32, device=ref.device)
    rc = load_library().cpmtp_verify_draft(N, n, _ptr(draft), _ptr(base_tokens), _ptr(logp_prefix), _ptr(logp_base),
                                           _ptr(uniform), _ptr(accepted), _stream())
    _check(rc)
    return accepted


def score_draft_static(h, W_head, E, W_g, draft, *, want_prefix: bool = True,
                       dev_status: Optional[torch.Tensor] = None, out: Optional[dict] = None) -> dict:
    """cpmtp_score_draft_static: draft scoring for callers that cannot provide scratch memory.

    Same results as score_draft, but the library's built-in fixed scratch array is used instead
    of a workspace, so no device memory is requested from anyone; the output tensors are the
    only thing this wrapper creates, and only when `out` does not already hold them.  Shapes
    needing more than STATIC_SCRATCH_BYTES raise CpmtpError (code -7).  Calls share the array:
    do not let two of them overlap on the GPU.
    """
    lib = load_library()
    shape = _shape_of(h, W_head, E, W_g, draft, None)
    res = out if out is not None else {}
    if "logp_joint" not in res:
        res["logp_joint"] = torch.empty(shape.N, dtype=torch.float32, device=h.device)
    if want_prefix and "logp_prefix" not in res:
        res["logp_prefix"] = torch.empty((shape.N, shape.n), dtype=torch.float32, device=h.device)
    rc = lib.cpmtp_score_draft_static(ctypes.byref(shape), _ptr(h), _ptr(W_head), _ptr(E), _ptr(W_g), _ptr(draft),
                                      _ptr(res["logp_joint"]), _ptr(res.get("logp_prefix")) if want_prefix else None,
                                      _ptr(dev_status), _stream())
    _check(rc)
    return res


def forward_host(h_host, W_head, E, W_g, x_host, logp_host, loss_host, *, aux_coef: Optional[float] = None,
                 saved: Optional[Saved] = None, workspace: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None) -> None:
    """cpmtp_forward_host: h_host / x_host / logp_host / loss_host are (pinned) CPU tensors; weights on device.
    Asynchronous: synchronise the current stream before reading the host outputs."""
    lib = load_library()
    N, d = h_host.shape
    shape = make_shape(N, d, E.shape[0], x_host.shape[1], W_g.shape[0], aux_coef)
    need = workspace_bytes(shape, OP_FORWARD) + host_staging_bytes(shape) + 256
    if workspace is None:
        workspace = alloc_workspace(need, E.device)
    cs = saved.c_struct() if saved is not None else None
    rc = lib.cpmtp_forward_host(ctypes.byref(shape), _ptr(h_host), _ptr(W_head), _ptr(E), _ptr(W_g), _ptr(x_host),
                                _ptr(logp_host), _ptr(loss_host), ctypes.byref(cs) if cs is not None else None,
                                _ptr(workspace), workspace.numel(),
                                _ptr(dev_status), _stream())
    _check(rc)


@dataclass
class DistillSaved:
    """Results of cpmtp_distill_forward kept for cpmtp_distill_backward (device tensors); `kl` is also
    the entry point's output, KL(p^d_k, p^c_k) per (position, token)."""
    lse_t: torch.Tensor
    logpi: torch.Tensor
    pm: torch.Tensor
    kl: torch.Tensor

    @staticmethod
    def alloc(shape: CShape, device="cuda") -> "DistillSaved":
        f = dict(dtype=torch.float32, device=device)
        K = shape.n * shape.r
        return DistillSaved(lse_t=torch.empty((shape.N, shape.n), **f), logpi=torch.empty((shape.N, K), **f),
                            pm=torch.empty((shape.N, K), **f), kl=torch.empty((shape.N, shape.n), **f))

    def c_struct(self) -> CDistillSaved:
        return CDistillSaved(self.lse_t.data_ptr(), self.logpi.data_ptr(), self.pm.data_ptr(), self.kl.data_ptr())


def _check_teacher(teacher, shape: CShape) -> None:
    assert teacher.shape == (shape.N, shape.n, shape.V) and teacher.dtype == torch.bfloat16 and teacher.is_contiguous()


def distill_forward(h, W_head, E, W_g, x, teacher, saved: Saved, dsaved: DistillSaved, *, beta: float = 0.9,
                    gamma: float = 1.0, aux_coef: Optional[float] = None, want_loss: bool = True,
                    workspace: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                    out: Optional[dict] = None, recompute_z: bool = False) -> dict:
    """cpmtp_distill_forward; returns {"logp", "logp_prefix", "kl", "loss"} (device tensors; kl is dsaved.kl)."""
    lib = load_library()
    shape = _shape_of(h, W_head, E, W_g, x, aux_coef)
    _check_teacher(teacher, shape)
    if recompute_z:
        shape.flags |= FLAG_RECOMPUTE_Z
    dev = h.device
    if workspace is None:
        workspace = alloc_workspace(workspace_bytes(shape, OP_DISTILL_FORWARD), dev)
    res = out if out is not None else {}
    res.setdefault("logp", torch.empty(shape.N, dtype=torch.float32, device=dev))
    res.setdefault("logp_prefix", torch.empty((shape.N, shape.n), dtype=torch.float32, device=dev))
    if want_loss:
        res.setdefault("loss", torch.empty(1, dtype=torch.float32, device=dev))
    res["kl"] = dsaved.kl
    cs, ds = saved.c_struct(), dsaved.c_struct()
    rc = lib.cpmtp_distill_forward(ctypes.byref(shape), _ptr(h), _ptr(W_head), _ptr(E), _ptr(W_g), _ptr(x),
                                   _ptr(teacher), ctypes.c_float(beta), ctypes.c_float(gamma), _ptr(res["logp"]),
                                   _ptr(res["logp_prefix"]), _ptr(res.get("loss")) if want_loss else None,
                                   ctypes.byref(cs), ctypes.byref(ds), _ptr(workspace), workspace.numel(),
                                   _ptr(dev_status), _stream())
    _check(rc)
    return res


def distill_backward(h, W_head, E, W_g, x, teacher, saved: Saved, dsaved: DistillSaved, *, beta: float = 0.9,
                     gamma: float = 1.0, aux_coef: Optional[float] = None,
                     dloss_dprefix: Optional[torch.Tensor] = None, dloss_dkl: Optional[torch.Tensor] = None,
                     workspace: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                     out: Optional[dict] = None, skip: tuple = (), recompute_z: bool = False,
                     accumulate: bool = False) -> dict:
    """cpmtp_distill_backward; returns {"dh", "dW_head", "dE", "dW_g"} (bf16 device tensors)."""
    lib = load_library()
    shape = _shape_of(h, W_head, E, W_g, x, aux_coef)
    _check_teacher(teacher, shape)
    if recompute_z:
        shape.flags |= FLAG_RECOMPUTE_Z
    if accumulate:
        assert out is not None, "accumulation needs the tensors to add to"
        shape.flags |= FLAG_ACCUM_GRADS
    for w in (dloss_dprefix, dloss_dkl):
        assert w is None or (w.shape == (shape.N, shape.n) and w.dtype == torch.float32 and w.is_contiguous())
    if workspace is None:
        workspace = alloc_workspace(workspace_bytes(shape, OP_DISTILL_BACKWARD), h.device)
    res = out if out is not None else {}
    for name, ref in (("dh", h), ("dW_head", W_head), ("dE", E), ("dW_g", W_g)):
        if name not in res and name not in skip:
            res[name] = torch.empty_like(ref)
    cs, ds = saved.c_struct(), dsaved.c_struct()
    rc = lib.cpmtp_distill_backward(ctypes.byref(shape), _ptr(h), _ptr(W_head), _ptr(E), _ptr(W_g), _ptr(x),
                                    _ptr(teacher), ctypes.byref(cs), ctypes.byref(ds), ctypes.c_float(beta),
                                    ctypes.c_float(gamma), _ptr(dloss_dprefix), _ptr(dloss_dkl), _ptr(res.get("dh")),
                                    _ptr(res.get("dW_head")), _ptr(res.get("dE")), _ptr(res.get("dW_g")),
                                    _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream())
    _check(rc)
    return res
