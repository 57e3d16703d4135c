"""ctypes binding of libha_la.so: argument marshalling only, same names as include/ha_la.h.

Every step of the prefill runs in the library's CUDA kernels.  There is no CPU or
PyTorch fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

HA_LA_GDN, HA_LA_KDA = 0, 1
HA_LA_BF16, HA_LA_FP32 = 0, 1
HA_LA_OK = 0
HA_LA_ERR_INVALID_ARG = 1
HA_LA_ERR_UNSUPPORTED = 2
HA_LA_ERR_WORKSPACE = 3
HA_LA_ERR_CUDA = 4
HA_LA_ERR_TIMEOUT = 5
HA_LA_ERR_DEVICE_CHECK = 6
HA_LA_ERR_TOO_LARGE = 7

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libha_la.so")

EXPORTS = (
    "ha_la_prefill_workspace_bytes",
    "ha_la_prefill",
    "ha_la_prefill_timed",
    "ha_la_prefill_noalloc",
    "ha_la_prefill_noalloc_scratch_bytes",
    "ha_la_prefill_path",
    "ha_la_prefill_num_launches",
    "ha_la_prefill_launch_plan",
    "ha_la_prefill_num_segments",
    "ha_la_decode",
    "ha_la_debug_wait_timeout",
    "ha_la_status_string",
    "ha_la_version",
)


class ha_la_prefill_args(ctypes.Structure):
    _fields_ = [
        ("variant", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("batch", ctypes.c_int32),
        ("seqlen", ctypes.c_int32),
        ("num_qk_heads", ctypes.c_int32),
        ("num_v_heads", ctypes.c_int32),
        ("d_k", ctypes.c_int32),
        ("d_v", ctypes.c_int32),
        ("chunk", ctypes.c_int32),
        ("scale", ctypes.c_float),
        ("q", ctypes.c_void_p),
        ("k", ctypes.c_void_p),
        ("v", ctypes.c_void_p),
        ("g", ctypes.c_void_p),
        ("beta", ctypes.c_void_p),
        ("h0", ctypes.c_void_p),
        ("cu_seqlens", ctypes.c_void_p),
        ("num_seqs", ctypes.c_int32),
        ("max_seqlen", ctypes.c_int32),
        ("o", ctypes.c_void_p),
        ("hT", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t),
        ("status_word", ctypes.c_void_p),
    ]


class ha_la_decode_args(ctypes.Structure):
    _fields_ = [
        ("variant", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("num_seqs", ctypes.c_int32),
        ("num_qk_heads", ctypes.c_int32),
        ("num_v_heads", ctypes.c_int32),
        ("d_k", ctypes.c_int32),
        ("d_v", ctypes.c_int32),
        ("scale", ctypes.c_float),
        ("q", ctypes.c_void_p),
        ("k", ctypes.c_void_p),
        ("v", ctypes.c_void_p),
        ("g", ctypes.c_void_p),
        ("beta", ctypes.c_void_p),
        ("h_in", ctypes.c_void_p),
        ("h_out", ctypes.c_void_p),
        ("o", ctypes.c_void_p),
    ]


class HaLaError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


_lib = None


def load_library(path: Optional[str] = None):
    """Load libha_la.so (built in-tree by paper_2609_32114_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(
            f"{p} not found: build it with `python -m paper_2609_32114_b200.build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(p)
    A = ctypes.POINTER(ha_la_prefill_args)
    lib.ha_la_prefill_workspace_bytes.argtypes = [A, ctypes.POINTER(ctypes.c_size_t)]
    lib.ha_la_prefill_workspace_bytes.restype = ctypes.c_int
    lib.ha_la_prefill.argtypes = [A, ctypes.c_void_p]
    lib.ha_la_prefill.restype = ctypes.c_int
    lib.ha_la_prefill_timed.argtypes = [A, ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_float),
                                        ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_int)]
    lib.ha_la_prefill_timed.restype = ctypes.c_int
    lib.ha_la_prefill_noalloc.argtypes = [A, ctypes.c_void_p]
    lib.ha_la_prefill_noalloc.restype = ctypes.c_int
    lib.ha_la_prefill_noalloc_scratch_bytes.argtypes = []
    lib.ha_la_prefill_noalloc_scratch_bytes.restype = ctypes.c_size_t
    lib.ha_la_prefill_path.argtypes = [A]
    lib.ha_la_prefill_path.restype = ctypes.c_char_p
    lib.ha_la_prefill_num_launches.argtypes = [A]
    lib.ha_la_prefill_num_launches.restype = ctypes.c_int
    lib.ha_la_prefill_num_segments.argtypes = [A]
    lib.ha_la_prefill_num_segments.restype = ctypes.c_int
    lib.ha_la_prefill_launch_plan.argtypes = [A, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int)]
    lib.ha_la_prefill_launch_plan.restype = ctypes.c_int
    lib.ha_la_decode.argtypes = [ctypes.POINTER(ha_la_decode_args), ctypes.c_void_p]
    lib.ha_la_decode.restype = ctypes.c_int
    lib.ha_la_debug_wait_timeout.argtypes = [A, ctypes.c_void_p, ctypes.c_uint]
    lib.ha_la_debug_wait_timeout.restype = ctypes.c_int
    lib.ha_la_status_string.argtypes = [ctypes.c_int]
    lib.ha_la_status_string.restype = ctypes.c_char_p
    lib.ha_la_version.argtypes = []
    lib.ha_la_version.restype = ctypes.c_int
    if path is None:
        _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().ha_la_status_string(int(status)).decode()


def ha_la_version() -> int:
    return load_library().ha_la_version()


def make_args(*, variant, dtype, batch, seqlen, hk, hv, dk, dv, scale=1.0, chunk=64, num_seqs=0, max_seqlen=0,
              q=0, k=0, v=0, g=0, beta=0, h0=0, cu_seqlens=0, o=0, hT=0, workspace=0, workspace_bytes=0,
              status_word=0) -> ha_la_prefill_args:
    """Fill the C struct from plain integers (device addresses) and sizes."""
    var = {"gdn": HA_LA_GDN, "kda": HA_LA_KDA}.get(variant, variant)
    dt = {"bf16": HA_LA_BF16, "fp32": HA_LA_FP32}.get(dtype, dtype)
    n = lambda p: p if p else None
    return ha_la_prefill_args(var, dt, batch, seqlen, hk, hv, dk, dv, chunk, float(scale), n(q), n(k), n(v), n(g),
                              n(beta), n(h0), n(cu_seqlens), num_seqs, max_seqlen, n(o), n(hT), n(workspace),
                              workspace_bytes, n(status_word))


def ha_la_prefill_workspace_bytes(args: ha_la_prefill_args) -> int:
    out = ctypes.c_size_t(0)
    rc = load_library().ha_la_prefill_workspace_bytes(ctypes.byref(args), ctypes.byref(out))
    if rc != HA_LA_OK:
        raise HaLaError(rc, "ha_la_prefill_workspace_bytes")
    return out.value


def ha_la_prefill_path(args: ha_la_prefill_args) -> Optional[str]:
    r = load_library().ha_la_prefill_path(ctypes.byref(args))
    return None if r is None else r.decode()


def ha_la_prefill_num_launches(args: ha_la_prefill_args) -> int:
    return load_library().ha_la_prefill_num_launches(ctypes.byref(args))


def ha_la_prefill_num_segments(args: ha_la_prefill_args) -> int:
    """Segments a sequence's chunks are cut into (1 = walked strictly in order)."""
    return load_library().ha_la_prefill_num_segments(ctypes.byref(args))


def ha_la_prefill_launch_plan(args: ha_la_prefill_args) -> Tuple[int, bool]:
    """(slice width of the sequential kernel or 0 on the CUDA-core path, kernels side by side?)."""
    nv, conc = ctypes.c_int(0), ctypes.c_int(0)
    rc = load_library().ha_la_prefill_launch_plan(ctypes.byref(args), ctypes.byref(nv), ctypes.byref(conc))
    if rc != HA_LA_OK:
        raise HaLaError(rc, "ha_la_prefill_launch_plan")
    return nv.value, bool(conc.value)


def ha_la_prefill_raw(args: ha_la_prefill_args, stream: int = 0) -> int:
    """The C call itself; returns the status code."""
    return load_library().ha_la_prefill(ctypes.byref(args), ctypes.c_void_p(stream) if stream else None)


def ha_la_prefill_noalloc(args: ha_la_prefill_args, stream: int = 0) -> int:
    """The C call for callers that cannot supply scratch memory (the workspace fields are ignored);
    returns the status code.  See include/ha_la.h for its limits and its sharing rules."""
    return load_library().ha_la_prefill_noalloc(ctypes.byref(args), ctypes.c_void_p(stream) if stream else None)


def ha_la_debug_wait_timeout(args: ha_la_prefill_args, stream: int = 0, spin_limit: int = 4096) -> int:
    """Test hook: the sequential kernel alone, waiting for flags nothing publishes; returns the status code."""
    return load_library().ha_la_debug_wait_timeout(ctypes.byref(args), ctypes.c_void_p(stream) if stream else None,
                                                   ctypes.c_uint(spin_limit))


def ha_la_prefill_noalloc_scratch_bytes() -> int:
    return load_library().ha_la_prefill_noalloc_scratch_bytes()


def ha_la_prefill_timed(args: ha_la_prefill_args, stream: int = 0):
    """Blocking, per-kernel device timing.  Returns [(kernel name, milliseconds), ...] in launch order."""
    ms = (ctypes.c_float * 8)()
    names = (ctypes.c_char_p * 8)()
    n = ctypes.c_int(0)
    rc = load_library().ha_la_prefill_timed(ctypes.byref(args), ctypes.c_void_p(stream) if stream else None, 8, ms,
                                            names, ctypes.byref(n))
    if rc != HA_LA_OK:
        raise HaLaError(rc, "ha_la_prefill_timed")
    return [(names[i].decode(), float(ms[i])) for i in range(n.value)]


def prepare_args(q, k, v, g, beta, *, variant="gdn", h0=None, cu_seqlens=None, max_seqlen=0, scale=1.0,
                 o=None, hT=None, want_hT=True, workspace=None, status_word=None):
    """Marshal torch CUDA tensors into ha_la_prefill_args (allocating o / hT / workspace / status word
    with torch when they are not given).  Returns (args, tensors) where `tensors` keeps them alive."""
    import torch

    if not q.is_cuda:
        raise ValueError("ha_la_prefill needs CUDA tensors (there is no CPU path)")
    packed = cu_seqlens is not None
    if q.dim() == 3:
        q, k, v, g, beta = (t.unsqueeze(0) for t in (q, k, v, g, beta))
        if o is not None:
            o = o.unsqueeze(0)
    B, T, HK, dk = q.shape
    HV, dv = v.shape[2], v.shape[3]
    dtype = {torch.bfloat16: "bf16", torch.float32: "fp32"}[q.dtype]
    for t in (q, k, v, g, beta):
        assert t.is_contiguous()
    assert k.dtype == q.dtype and v.dtype == q.dtype and g.dtype == torch.float32 and beta.dtype == torch.float32
    N = (cu_seqlens.numel() - 1) if packed else B
    if packed:
        assert cu_seqlens.dtype == torch.int32 and cu_seqlens.is_cuda and B == 1
    if o is None:
        o = torch.empty_like(v)
    if hT is None and want_hT:
        hT = torch.empty((N, HV, dk, dv), dtype=torch.float32, device=q.device)
    if status_word is None:
        status_word = torch.zeros(1, dtype=torch.int32, device=q.device)
    ptr = lambda t: 0 if t is None else t.data_ptr()
    args = make_args(variant=variant, dtype=dtype, batch=B, seqlen=T, hk=HK, hv=HV, dk=dk, dv=dv, scale=scale,
                     num_seqs=N if packed else 0, max_seqlen=max_seqlen, q=ptr(q), k=ptr(k), v=ptr(v), g=ptr(g),
                     beta=ptr(beta), h0=ptr(h0), cu_seqlens=ptr(cu_seqlens), o=ptr(o), hT=ptr(hT),
                     status_word=ptr(status_word))
    need = ha_la_prefill_workspace_bytes(args)
    if workspace is None:
        workspace = torch.empty(need + 256, dtype=torch.uint8, device=q.device)
    wp = (workspace.data_ptr() + 255) // 256 * 256
    args.workspace = wp
    args.workspace_bytes = workspace.numel() - (wp - workspace.data_ptr())
    keep = dict(q=q, k=k, v=v, g=g, beta=beta, h0=h0, cu_seqlens=cu_seqlens, o=o, hT=hT, workspace=workspace,
                status_word=status_word)
    return args, keep


def ha_la_prefill(q, k, v, g, beta, *, stream=None, **kw):
    """Prefill on torch CUDA tensors: prepare_args + the C call on torch's current stream.

    q, k : [B, T, HK, dk] (or [T, HK, dk])   v : [B, T, HV, dv]   bf16 or fp32
    g    : fp32 [B, T, HV] (gdn) or [B, T, HV, dk] (kda)      beta : fp32 [B, T, HV]
    h0   : fp32 [N, HV, dk, dv] or None      cu_seqlens : int32 [N+1] device tensor or None (packed, B = 1)
    Returns (o, hT, status_word, workspace); nothing is synchronised.
    """
    import torch

    squeeze = q.dim() == 3
    args, keep = prepare_args(q, k, v, g, beta, **kw)
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    rc = ha_la_prefill_raw(args, stream)
    if rc != HA_LA_OK:
        raise HaLaError(rc, "ha_la_prefill")
    o = keep["o"].squeeze(0) if squeeze else keep["o"]
    return o, keep["hT"], keep["status_word"], keep["workspace"]


def prepare_decode_args(q, k, v, g, beta, state, *, variant="gdn", scale=1.0, o=None, state_out=None):
    """Marshal torch CUDA tensors into ha_la_decode_args.  q, k: [N, HK, d]; v: [N, HV, d]; g: fp32 [N, HV] (gdn)
    or [N, HV, d] (kda); beta: fp32 [N, HV]; state: fp32 [N, HV, d, d] or None (zeros).  The new state goes to
    `state_out` (default: in place into `state`; allocated when `state` is None)."""
    import torch

    N, HK, d = q.shape
    HV = v.shape[1]
    if o is None:
        o = torch.empty_like(v)
    if state_out is None:
        state_out = state if state is not None else torch.empty(N, HV, d, d, dtype=torch.float32, device=q.device)
    ptr = lambda t: t.data_ptr() if t is not None else None
    args = ha_la_decode_args(variant=0 if variant == "gdn" else 1, dtype=0 if q.dtype == torch.bfloat16 else 1,
                             num_seqs=N, num_qk_heads=HK, num_v_heads=HV, d_k=d, d_v=v.shape[2], scale=scale,
                             q=ptr(q), k=ptr(k), v=ptr(v), g=ptr(g), beta=ptr(beta), h_in=ptr(state),
                             h_out=ptr(state_out), o=ptr(o))
    return args, dict(q=q, k=k, v=v, g=g, beta=beta, state=state, state_out=state_out, o=o)


def ha_la_decode_raw(args: ha_la_decode_args, stream: int = 0) -> int:
    return load_library().ha_la_decode(ctypes.byref(args), ctypes.c_void_p(stream))


def ha_la_decode(q, k, v, g, beta, state, *, stream=None, **kw):
    """One decoding step on torch CUDA tensors (see prepare_decode_args).  Returns (o, new_state); nothing is
    synchronised."""
    import torch

    args, keep = prepare_decode_args(q, k, v, g, beta, state, **kw)
    if stream is None:
        stream = torch.cuda.current_stream(q.device).cuda_stream
    rc = ha_la_decode_raw(args, stream)
    if rc != HA_LA_OK:
        raise HaLaError(rc, "ha_la_decode")
    return keep["o"], keep["state_out"]
