"""ctypes binding of librdk_b200.so: argument marshalling only.

Every function below has the name of the C entry point it calls (see include/rdk.h), takes torch
tensors for the device buffers, and passes their data pointers and the current CUDA stream through.
All arithmetic runs in the CUDA kernels of the library.  There is no fallback: if the shared library
cannot be loaded, or a call returns an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, Optional

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "librdk_b200.so")

RDK_OK = 0
RDK_ERR_INVALID_ARG, RDK_ERR_BAD_IDS, RDK_ERR_EMPTY_INTERSECTION, RDK_ERR_UNSUPPORTED = 1, 2, 3, 4
RDK_ERR_WORKSPACE_TOO_SMALL, RDK_ERR_ARCH, RDK_ERR_CUDA, RDK_ERR_TIMEOUT = 5, 6, 7, 8
RDK_F32, RDK_BF16 = 0, 1
RDK_LOGITS, RDK_PROBS = 0, 1
RDK_MODE_LINEAR, RDK_MODE_PRECOMPUTED_W = 0, 1
RDK_AFF_F32_ROWS, RDK_AFF_BF16_COLS = 0, 1
RDK_FLAG_ROW_KERNEL = 1
RDK_FLAG_W_AS_GIVEN = 2
RDK_ROUTE_ROW_KERNEL, RDK_ROUTE_STREAM_KERNEL = 0, 1

EXPORTS = [
    "rdk_version", "rdk_status_string", "rdk_last_error", "rdk_kept_index_bytes", "rdk_prepare_ids",
    "rdk_build_affinity_workspace_bytes", "rdk_build_affinity", "rdk_exact_workspace_bytes",
    "rdk_redistribute_exact", "rdk_redistribute_exact_static", "rdk_redistribute_linear",
    "rdk_sample_workspace_bytes", "rdk_sample_and_verify", "rdk_emit_sequences",
    "rdk_sample_and_verify_host", "rdk_stream_geometry", "rdk_sample_and_verify_prior",
    "rdk_redistribute_linear_prior", "rdk_sample_route", "rdk_test_set_spin_limit",
]


class RdkError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str):
        super().__init__(f"{where}: status {status} ({detail})")
        self.status = status


class rdk_problem(C.Structure):
    _fields_ = [("N", C.c_int32), ("n", C.c_int32), ("batch", C.c_int32), ("positions", C.c_int32),
                ("target_dtype", C.c_int32), ("drafter_dtype", C.c_int32), ("drafter_kind", C.c_int32),
                ("flags", C.c_int32), ("target_row_stride", C.c_int64),
                ("drafter_row_stride", C.c_int64), ("kept_index", C.c_void_p)]


class rdk_affinity(C.Structure):
    _fields_ = [("data", C.c_void_p), ("layout", C.c_int32), ("reserved", C.c_int32), ("ld", C.c_int64)]


class rdk_stream_geometry_t(C.Structure):
    _fields_ = [("supported", C.c_int32), ("ctas_per_row", C.c_int32), ("warps_per_cta", C.c_int32),
                ("segment_tokens", C.c_int32), ("stages", C.c_int32), ("live_rows", C.c_int32),
                ("cached_slots_per_warp", C.c_int32), ("reserved", C.c_int32), ("dynamic_shared_bytes", C.c_int64)]


class rdk_outputs(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in
                ("draft_token", "out_token", "accepted", "accept_prob", "alpha", "theta", "S",
                 "residual_mass", "accepted_len", "status_word")]


_lib = None


def lib() -> C.CDLL:
    """Load the shared library (once).  Raises if it is missing: there is no other code path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2506_03206_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.rdk_version.restype = C.c_int
        L.rdk_status_string.restype = C.c_char_p
        L.rdk_status_string.argtypes = [C.c_int]
        L.rdk_last_error.restype = C.c_char_p
        L.rdk_kept_index_bytes.restype = C.c_size_t
        L.rdk_kept_index_bytes.argtypes = [C.c_int32, C.c_int32]
        L.rdk_prepare_ids.restype = C.c_int
        L.rdk_prepare_ids.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t,
                                      C.POINTER(C.c_int), C.c_void_p]
        L.rdk_build_affinity_workspace_bytes.restype = C.c_size_t
        L.rdk_build_affinity_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
        L.rdk_build_affinity.restype = C.c_int
        L.rdk_build_affinity.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int64, C.c_void_p, C.c_int32,
                                         C.c_int32, C.c_float, C.POINTER(rdk_affinity), C.c_void_p,
                                         C.c_void_p, C.c_size_t, C.c_void_p]
        L.rdk_exact_workspace_bytes.restype = C.c_size_t
        L.rdk_exact_workspace_bytes.argtypes = [C.POINTER(rdk_problem), C.c_int32]
        L.rdk_redistribute_exact.restype = C.c_int
        L.rdk_redistribute_exact.argtypes = [C.POINTER(rdk_problem), C.c_void_p, C.POINTER(rdk_affinity),
                                             C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p,
                                             C.c_void_p]
        L.rdk_redistribute_exact_static.restype = C.c_int
        L.rdk_redistribute_exact_static.argtypes = [C.POINTER(rdk_problem), C.c_void_p, C.POINTER(rdk_affinity),
                                                    C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.rdk_redistribute_linear.restype = C.c_int
        L.rdk_redistribute_linear.argtypes = [C.POINTER(rdk_problem), C.c_void_p, C.c_void_p, C.c_void_p,
                                              C.c_void_p, C.c_void_p, C.c_void_p]
        L.rdk_sample_and_verify.restype = C.c_int
        L.rdk_sample_and_verify.argtypes = [C.POINTER(rdk_problem), C.c_int32, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_int64, C.c_void_p, C.c_int32,
                                            C.POINTER(rdk_outputs), C.c_void_p, C.c_size_t, C.c_void_p]
        L.rdk_sample_workspace_bytes.restype = C.c_size_t
        L.rdk_sample_workspace_bytes.argtypes = [C.POINTER(rdk_problem), C.c_int32, C.c_int32]
        L.rdk_emit_sequences.restype = C.c_int
        L.rdk_emit_sequences.argtypes = [C.POINTER(rdk_problem), C.c_void_p, C.c_int64, C.c_void_p, C.c_int32,
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.rdk_sample_and_verify_host.restype = C.c_int
        L.rdk_sample_and_verify_host.argtypes = [C.POINTER(rdk_problem), C.c_void_p, C.c_void_p, C.c_void_p,
                                                 C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                                 C.POINTER(rdk_outputs), C.POINTER(rdk_outputs), C.c_void_p,
                                                 C.c_size_t, C.c_void_p]
        L.rdk_sample_route.restype = C.c_int
        L.rdk_sample_route.argtypes = [C.POINTER(rdk_problem), C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                       C.c_void_p, C.c_size_t, C.POINTER(C.c_char_p)]
        L.rdk_test_set_spin_limit.restype = None
        L.rdk_test_set_spin_limit.argtypes = [C.c_uint32]
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != RDK_OK:
        L = lib()
        raise RdkError(status, where, f"{L.rdk_status_string(status).decode()}: {L.rdk_last_error().decode()}")


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return RDK_F32
    if t.dtype == torch.bfloat16:
        return RDK_BF16
    raise TypeError(f"unsupported dtype {t.dtype}: the library takes float32 or bfloat16")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _rows2d(t: torch.Tensor, what: str) -> None:
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError(f"{what} must be 2-D with contiguous rows")


@dataclass
class KeptIndex:
    """Device-side index of the kept ids, filled by rdk_prepare_ids."""
    buffer: torch.Tensor
    N: int
    n: int
    n_valid: int


def rdk_version() -> int:
    return lib().rdk_version()


def rdk_prepare_ids(kept_ids: torch.Tensor, N: int) -> KeptIndex:
    if kept_ids.dtype != torch.int32 or kept_ids.dim() != 1 or not kept_ids.is_contiguous():
        raise TypeError("kept_ids must be a contiguous 1-D int32 tensor")
    n = kept_ids.numel()
    nbytes = lib().rdk_kept_index_bytes(N, n)
    if nbytes == 0:
        raise RdkError(RDK_ERR_INVALID_ARG, "rdk_kept_index_bytes", f"N={N} n={n}")
    buf = torch.empty(nbytes, dtype=torch.uint8, device=kept_ids.device)
    nv = C.c_int(0)
    _check(lib().rdk_prepare_ids(kept_ids.data_ptr(), n, N, buf.data_ptr(), nbytes, C.byref(nv), _stream()),
           "rdk_prepare_ids")
    return KeptIndex(buf, N, n, nv.value)


def make_problem(index: KeptIndex, target: Optional[torch.Tensor], drafter: Optional[torch.Tensor],
                 batch: int, positions: int, drafter_kind: int = RDK_LOGITS,
                 target_dtype: Optional[int] = None, drafter_dtype: Optional[int] = None, flags: int = 0) -> rdk_problem:
    p = rdk_problem()
    p.N, p.n, p.batch, p.positions = index.N, index.n, batch, positions
    p.target_dtype = _dtype_code(target) if target is not None else (target_dtype or RDK_F32)
    p.drafter_dtype = _dtype_code(drafter) if drafter is not None else (drafter_dtype or RDK_F32)
    p.drafter_kind = drafter_kind
    p.flags = flags
    p.target_row_stride = target.stride(0) if target is not None else 0
    p.drafter_row_stride = drafter.stride(0) if drafter is not None else 0
    p.kept_index = index.buffer.data_ptr()
    return p


def affinity_alloc(N: int, n: int, layout: int, device) -> Dict[str, object]:
    """Allocate an affinity matrix in one of the two layouts of rdk_affinity_layout."""
    if layout == RDK_AFF_F32_ROWS:
        data = torch.zeros(n, N, dtype=torch.float32, device=device)
        ld = N
    else:
        ld = (n + 7) // 8 * 8
        data = torch.zeros(N, ld, dtype=torch.bfloat16, device=device)
    return {"data": data, "layout": layout, "ld": ld}


def _aff_struct(M: Dict[str, object]) -> rdk_affinity:
    a = rdk_affinity()
    a.data, a.layout, a.reserved, a.ld = M["data"].data_ptr(), M["layout"], 0, M["ld"]
    return a


def rdk_build_affinity(embeddings: torch.Tensor, kept_ids: torch.Tensor, tau: float, layout: int) -> Dict[str, object]:
    _rows2d(embeddings, "embeddings")
    N, d = embeddings.shape
    n = kept_ids.numel()
    M = affinity_alloc(N, n, layout, embeddings.device)
    wsb = lib().rdk_build_affinity_workspace_bytes(N, n, d)
    ws = torch.empty(wsb, dtype=torch.uint8, device=embeddings.device)
    a = _aff_struct(M)
    _check(lib().rdk_build_affinity(embeddings.data_ptr(), _dtype_code(embeddings), d, embeddings.stride(0),
                                    kept_ids.data_ptr(), n, N, float(tau), C.byref(a), M["data"].data_ptr(),
                                    ws.data_ptr(), wsb, _stream()), "rdk_build_affinity")
    M["_ws"] = ws      # keep the workspace alive until the stream has consumed it
    return M


def rdk_redistribute_exact(index: KeptIndex, drafter: torch.Tensor, M: Dict[str, object], batch: int,
                           positions: int, drafter_kind: int = RDK_LOGITS,
                           w_out: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None,
                           status_word: Optional[torch.Tensor] = None):
    _rows2d(drafter, "drafter")
    rows = batch * positions
    pb = make_problem(index, None, drafter, batch, positions, drafter_kind)
    if w_out is None:
        w_out = torch.empty(rows, index.N, dtype=torch.float32, device=drafter.device)
    S = torch.empty(rows, dtype=torch.float32, device=drafter.device)
    wsb = lib().rdk_exact_workspace_bytes(C.byref(pb), M["layout"])
    if ws is None:
        ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device=drafter.device)
    a = _aff_struct(M)
    _check(lib().rdk_redistribute_exact(C.byref(pb), drafter.data_ptr(), C.byref(a), w_out.data_ptr(),
                                        S.data_ptr(), ws.data_ptr(), ws.numel(), _ptr(status_word), _stream()),
           "rdk_redistribute_exact")
    return w_out, S, ws


RDK_STATIC_SCRATCH_BYTES = 4 << 20


def rdk_redistribute_exact_static(index: KeptIndex, drafter: torch.Tensor, M: Dict[str, object], batch: int,
                                  positions: int, w_out: torch.Tensor, S_out: torch.Tensor,
                                  drafter_kind: int = RDK_LOGITS, status_word: Optional[torch.Tensor] = None) -> None:
    """rdk_redistribute_exact without a workspace argument: the library stages the q' operand in its
    own fixed device array, so this call (and this wrapper) allocates nothing -- the caller passes
    the output tensors in.  Meant for callers that must not touch the device allocator."""
    _rows2d(drafter, "drafter")
    pb = make_problem(index, None, drafter, batch, positions, drafter_kind)
    a = _aff_struct(M)
    _check(lib().rdk_redistribute_exact_static(C.byref(pb), drafter.data_ptr(), C.byref(a), w_out.data_ptr(),
                                               S_out.data_ptr(), _ptr(status_word), _stream()),
           "rdk_redistribute_exact_static")


def rdk_redistribute_linear(index: KeptIndex, target: torch.Tensor, drafter: torch.Tensor, batch: int,
                            positions: int, drafter_kind: int = RDK_LOGITS):
    _rows2d(target, "target")
    _rows2d(drafter, "drafter")
    rows = batch * positions
    pb = make_problem(index, target, drafter, batch, positions, drafter_kind)
    qt = torch.empty(rows, index.N, dtype=torch.float32, device=target.device)
    theta = torch.empty(rows, dtype=torch.float32, device=target.device)
    S = torch.empty(rows, dtype=torch.float32, device=target.device)
    _check(lib().rdk_redistribute_linear(C.byref(pb), target.data_ptr(), drafter.data_ptr(), qt.data_ptr(),
                                         theta.data_ptr(), S.data_ptr(), _stream()), "rdk_redistribute_linear")
    return qt, theta, S


def alloc_outputs(rows: int, batch: int, trials: int, device) -> Dict[str, torch.Tensor]:
    rt = rows * trials
    return {
        "draft_token": torch.empty(rt, dtype=torch.int32, device=device),
        "out_token": torch.empty(rt, dtype=torch.int32, device=device),
        "accepted": torch.empty(rt, dtype=torch.uint8, device=device),
        "accept_prob": torch.empty(rt, dtype=torch.float32, device=device),
        "alpha": torch.empty(rows, dtype=torch.float32, device=device),
        "theta": torch.zeros(rows, dtype=torch.float32, device=device),
        "S": torch.empty(rows, dtype=torch.float32, device=device),
        "residual_mass": torch.empty(rows, dtype=torch.float32, device=device),
        "accepted_len": torch.empty(batch * trials, dtype=torch.int32, device=device),
        "status_word": torch.zeros(1, dtype=torch.int32, device=device),
    }


def outputs_struct(out: Dict[str, torch.Tensor]) -> rdk_outputs:
    o = rdk_outputs()
    for name, _ in rdk_outputs._fields_:
        setattr(o, name, _ptr(out.get(name)))   # absent members stay NULL
    return o


def sample_workspace(pb: rdk_problem, mode: int, trials: int, device) -> torch.Tensor:
    nbytes = lib().rdk_sample_workspace_bytes(C.byref(pb), mode, trials)
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def rdk_sample_and_verify(index: KeptIndex, mode: int, target: torch.Tensor,
                          drafter: Optional[torch.Tensor], w: Optional[torch.Tensor],
                          uniforms: torch.Tensor, batch: int, positions: int,
                          drafter_kind: int = RDK_LOGITS,
                          out: Optional[Dict[str, torch.Tensor]] = None,
                          ws: Optional[torch.Tensor] = None, flags: int = 0) -> Dict[str, torch.Tensor]:
    _rows2d(target, "target")
    rows = batch * positions
    if uniforms.dtype != torch.float32 or not uniforms.is_contiguous() or uniforms.numel() % (rows * 4):
        raise ValueError("uniforms must be contiguous float32 [rows, trials, 4]")
    trials = uniforms.numel() // (rows * 4)
    pb = make_problem(index, target, drafter, batch, positions, drafter_kind, flags=flags)
    if out is None:
        out = alloc_outputs(rows, batch, trials, target.device)
    o = outputs_struct(out)
    if ws is None:
        ws = sample_workspace(pb, mode, trials, target.device)
    _check(lib().rdk_sample_and_verify(C.byref(pb), mode, target.data_ptr(), _ptr(drafter), _ptr(w),
                                       0 if w is None else w.stride(0), uniforms.data_ptr(), trials,
                                       C.byref(o), ws.data_ptr(), ws.numel(), _stream()), "rdk_sample_and_verify")
    out["_ws"] = ws        # keep the workspace alive until the stream has consumed it
    return out


def rdk_sample_route(index: KeptIndex, mode: int, target: torch.Tensor, drafter: Optional[torch.Tensor],
                     batch: int, positions: int, trials: int, ws: Optional[torch.Tensor],
                     drafter_kind: int = RDK_LOGITS, flags: int = 0):
    """Host-only query: (route, reason) -- which kernel rdk_sample_and_verify would take for these arguments."""
    pb = make_problem(index, target, drafter, batch, positions, drafter_kind, flags=flags)
    why = C.c_char_p()
    r = lib().rdk_sample_route(C.byref(pb), mode, target.data_ptr(), _ptr(drafter), trials, _ptr(ws),
                               0 if ws is None else ws.numel(), C.byref(why))
    if r < 0:
        _check(-r, "rdk_sample_route")
    return r, (why.value or b"").decode()


def rdk_test_set_spin_limit(limit: int) -> None:
    """Tests of the failure path only: failed tries after which a device-side wait gives up (0 = default)."""
    lib().rdk_test_set_spin_limit(int(limit))


def rdk_emit_sequences(N: int, batch: int, positions: int, bonus_target: torch.Tensor, uniforms: torch.Tensor,
                       draft_token: torch.Tensor, accepted: torch.Tensor, out_token: torch.Tensor):
    """Returns (seq_tokens int32 [batch, trials, positions + 1], seq_len int32 [batch, trials])."""
    _rows2d(bonus_target, "bonus_target")
    trials = uniforms.numel() // (batch * positions * 4)
    pb = rdk_problem()
    pb.N, pb.n, pb.batch, pb.positions = N, 1, batch, positions
    pb.target_dtype = _dtype_code(bonus_target)
    seq = torch.full((batch, trials, positions + 1), -1, dtype=torch.int32, device=bonus_target.device)
    ln = torch.empty(batch, trials, dtype=torch.int32, device=bonus_target.device)
    _check(lib().rdk_emit_sequences(C.byref(pb), bonus_target.data_ptr(), bonus_target.stride(0), uniforms.data_ptr(),
                                    trials, draft_token.data_ptr(), accepted.data_ptr(), out_token.data_ptr(),
                                    seq.data_ptr(), ln.data_ptr(), _stream()), "rdk_emit_sequences")
    return seq, ln


def rdk_sample_and_verify_host(index: KeptIndex, target_host: torch.Tensor, drafter_host: torch.Tensor,
                               uniforms_host: torch.Tensor, batch: int, positions: int, stage: Dict[str, torch.Tensor],
                               dev_out: Dict[str, torch.Tensor], host_out: Dict[str, torch.Tensor],
                               drafter_kind: int = RDK_LOGITS) -> Dict[str, torch.Tensor]:
    """`stage` holds the device staging tensors "target", "drafter", "uniforms" and the workspace "ws"."""
    rows = batch * positions
    trials = uniforms_host.numel() // (rows * 4)
    pb = make_problem(index, stage["target"], stage["drafter"], batch, positions, drafter_kind)
    od, oh = outputs_struct(dev_out), outputs_struct(host_out)
    _check(lib().rdk_sample_and_verify_host(C.byref(pb), target_host.data_ptr(), drafter_host.data_ptr(),
                                            uniforms_host.data_ptr(), trials, stage["target"].data_ptr(),
                                            stage["drafter"].data_ptr(), stage["uniforms"].data_ptr(),
                                            C.byref(od), C.byref(oh), stage["ws"].data_ptr(), stage["ws"].numel(),
                                            _stream()), "rdk_sample_and_verify_host")
    return host_out


def check_status_word(out: Dict[str, torch.Tensor], where: str = "kernel") -> None:
    """Read the device status word (synchronises) and raise if a kernel reported an error."""
    code = int(out["status_word"].item())
    if code != 0:
        raise RdkError(code, where, lib().rdk_status_string(code).decode())


def rdk_stream_geometry(N: int, n: int, target_dtype: int = RDK_BF16, drafter_dtype: int = RDK_BF16) -> Dict[str, int]:
    """How the streaming kernels of the linear mode would lay out a problem (host-only query)."""
    L = lib()
    L.rdk_stream_geometry.restype = C.c_int
    L.rdk_stream_geometry.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(rdk_stream_geometry_t)]
    g = rdk_stream_geometry_t()
    _check(L.rdk_stream_geometry(N, n, target_dtype, drafter_dtype, C.byref(g)), "rdk_stream_geometry")
    return {k: int(getattr(g, k)) for k, _ in rdk_stream_geometry_t._fields_ if k != "reserved"}


def _prior_stride(prior: torch.Tensor, N: int) -> int:
    """A [N] prior is one row shared by all rows (stride 0); a [rows, N] prior has its row stride."""
    if prior.dim() == 1:
        if prior.numel() != N or not prior.is_contiguous():
            raise ValueError("a shared prior must be a contiguous [N] tensor")
        return 0
    _rows2d(prior, "prior")
    return prior.stride(0)


def rdk_redistribute_linear_prior(index: KeptIndex, target: torch.Tensor, prior: torch.Tensor, drafter: torch.Tensor,
                                  batch: int, positions: int, drafter_kind: int = RDK_LOGITS):
    """Eq. rdk-taylor with softmax(prior) in place of p, written out: (q~ [rows, N], theta, S)."""
    _rows2d(target, "target")
    _rows2d(drafter, "drafter")
    if prior.dtype != target.dtype:
        raise ValueError("the prior must have the target's dtype")
    rows = batch * positions
    pb = make_problem(index, target, drafter, batch, positions, drafter_kind)
    qt = torch.empty(rows, index.N, dtype=torch.float32, device=target.device)
    theta = torch.empty(rows, dtype=torch.float32, device=target.device)
    S = torch.empty(rows, dtype=torch.float32, device=target.device)
    L = lib()
    L.rdk_redistribute_linear_prior.restype = C.c_int
    L.rdk_redistribute_linear_prior.argtypes = [C.POINTER(rdk_problem), C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                                C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    _check(L.rdk_redistribute_linear_prior(C.byref(pb), target.data_ptr(), prior.data_ptr(), _prior_stride(prior, index.N),
                                           drafter.data_ptr(), qt.data_ptr(), theta.data_ptr(), S.data_ptr(), _stream()),
           "rdk_redistribute_linear_prior")
    return qt, theta, S


def rdk_sample_and_verify_prior(index: KeptIndex, target: torch.Tensor, prior: torch.Tensor, drafter: torch.Tensor,
                                uniforms: torch.Tensor, batch: int, positions: int, drafter_kind: int = RDK_LOGITS,
                                out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
    """The linear mode with a separate prior inside Eq. rdk-taylor; verification against softmax(target)."""
    _rows2d(target, "target")
    _rows2d(drafter, "drafter")
    if prior.dtype != target.dtype:
        raise ValueError("the prior must have the target's dtype")
    rows = batch * positions
    trials = uniforms.numel() // (rows * 4)
    pb = make_problem(index, target, drafter, batch, positions, drafter_kind)
    if out is None:
        out = alloc_outputs(rows, batch, trials, target.device)
    o = outputs_struct(out)
    L = lib()
    L.rdk_sample_and_verify_prior.restype = C.c_int
    L.rdk_sample_and_verify_prior.argtypes = [C.POINTER(rdk_problem), C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                              C.c_void_p, C.c_int32, C.POINTER(rdk_outputs), C.c_void_p]
    _check(L.rdk_sample_and_verify_prior(C.byref(pb), target.data_ptr(), prior.data_ptr(), _prior_stride(prior, index.N),
                                         drafter.data_ptr(), uniforms.data_ptr(), trials, C.byref(o), _stream()),
           "rdk_sample_and_verify_prior")
    return out
