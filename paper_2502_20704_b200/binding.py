"""ctypes binding of libfsd_verify.so.

The functions here carry the names and argument order of the C entry points and do
argument marshalling only: tensors become device pointers, the options become the C
struct.  There is no fallback: if the compiled library is missing, importing a
function from it raises.
"""

from __future__ import annotations

import ctypes as C
import os
from typing import Optional

_PKG = os.path.dirname(os.path.abspath(__file__))
# FSD_VERIFY_LIB selects another build of the same library (the debug build with range checks)
_LIB_PATH = os.environ.get("FSD_VERIFY_LIB") or os.path.join(_PKG, "lib", "libfsd_verify.so")

DIVS = {"js": 0, "kl": 1, "tv": 2}
MODES = {"fsd": 0, "sd": 1, "rfsd": 2}
CMPS = {"lt": 0, "le": 1}
SAMPLES = {"invcdf": 0, "greedy": 1}
DTYPES = {"f32": 0, "bf16": 1}

FSD_OK = 0
FSD_ERR_NULL, FSD_ERR_SHAPE, FSD_ERR_ALIGN, FSD_ERR_ENUM = -1, -2, -3, -4
FSD_ERR_WORKSPACE, FSD_ERR_UNSUPPORTED, FSD_ERR_CUDA, FSD_ERR_TOO_LARGE = -5, -6, -7, -8
FSD_STATIC_MAX_POSITIONS = 1024
FSD_ROW_NONFINITE, FSD_ROW_TIMEOUT, FSD_ROW_BADTREE = 1, 2, 4


class FsdOpts(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32),
        ("divergence", C.c_int32),
        ("mode", C.c_int32),
        ("compare", C.c_int32),
        ("sample", C.c_int32),
        ("logit_dtype", C.c_int32),
        ("threshold", C.c_float),
    ]


class FsdError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"fsd_verify failed: {fsd_status_string(status)} ({status})")


_lib = None


def library_path() -> str:
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2502_20704_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        lib = C.CDLL(_LIB_PATH)
        vp, ip, fp = C.c_void_p, C.c_void_p, C.c_void_p
        lib.fsd_default_opts.argtypes = [C.POINTER(FsdOpts)]
        lib.fsd_default_opts.restype = None
        lib.fsd_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int, C.POINTER(FsdOpts), C.POINTER(C.c_size_t)]
        lib.fsd_workspace_bytes.restype = C.c_int
        lib.fsd_verify_chain.argtypes = [vp, vp, ip, fp, fp, C.c_int, C.c_int, C.c_int, C.POINTER(FsdOpts),
                                         ip, ip, fp, ip, vp, C.c_size_t, vp]
        lib.fsd_verify_chain.restype = C.c_int
        lib.fsd_verify_tree.argtypes = [vp, vp, ip, fp, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(FsdOpts),
                                        ip, ip, ip, fp, ip, vp, C.c_size_t, vp]
        lib.fsd_verify_tree.restype = C.c_int
        lib.fsd_host_staging_bytes.argtypes = [C.c_int, C.c_int, C.c_int, C.POINTER(FsdOpts), C.POINTER(C.c_size_t)]
        lib.fsd_host_staging_bytes.restype = C.c_int
        lib.fsd_verify_chain_host.argtypes = [vp, vp, ip, fp, fp, C.c_int, C.c_int, C.c_int, C.POINTER(FsdOpts),
                                              ip, ip, fp, ip, vp, C.c_size_t, vp]
        lib.fsd_verify_chain_host.restype = C.c_int
        lib.fsd_verify_chain_static.argtypes = [vp, vp, ip, fp, fp, C.c_int, C.c_int, C.c_int, C.POINTER(FsdOpts),
                                                ip, ip, fp, ip, vp]
        lib.fsd_verify_chain_static.restype = C.c_int
        lib.fsd_status_string.argtypes = [C.c_int]
        lib.fsd_status_string.restype = C.c_char_p
        lib.fsd_version.restype = C.c_int
        lib.fsd_set_stage_event.argtypes = [C.c_void_p]
        lib.fsd_set_stage_event.restype = C.c_int
        lib.fsd_debug_checks.argtypes = [C.c_int, C.c_int, C.POINTER(C.c_size_t)]
        lib.fsd_debug_checks.restype = C.c_int
        lib.fsd_set_timeout_injection.argtypes = [C.c_int]
        lib.fsd_set_timeout_injection.restype = C.c_int
        lib.fsd_set_group_size.argtypes = [C.c_int]
        lib.fsd_set_group_size.restype = C.c_int
        lib.fsd_threshold_sweep.argtypes = [vp, C.c_int, C.c_int, vp, C.c_int, C.c_int, vp, vp, C.c_void_p]
        lib.fsd_threshold_sweep.restype = C.c_int
        lib.fsd_calibrate_threshold.argtypes = [vp, C.c_int, C.c_int, C.c_float, C.c_int, vp, vp, C.c_void_p]
        lib.fsd_calibrate_threshold.restype = C.c_int
        lib.fsd_accept_labels.argtypes = [vp, C.c_int, C.c_int, C.c_float, C.c_int, vp, C.c_void_p]
        lib.fsd_accept_labels.restype = C.c_int
        _lib = lib
    return _lib


def _ptr(t) -> Optional[int]:
    """Device (or raw integer) pointer of a tensor-like argument; None stays NULL."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def fsd_default_opts() -> FsdOpts:
    o = FsdOpts()
    _load().fsd_default_opts(C.byref(o))
    return o


def make_opts(div="js", mode="fsd", cmp="lt", sample="invcdf", dtype="bf16", T=0.0) -> FsdOpts:
    o = fsd_default_opts()
    o.divergence, o.mode, o.compare = DIVS[div], MODES[mode], CMPS[cmp]
    o.sample, o.logit_dtype, o.threshold = SAMPLES[sample], DTYPES[dtype], float(T)
    return o


def fsd_status_string(status: int) -> str:
    return _load().fsd_status_string(int(status)).decode()


def fsd_version() -> int:
    return _load().fsd_version()


def fsd_set_stage_event(event) -> int:
    """Record `event` (a ``torch.cuda.Event`` that has been created, a raw handle, or None) between
    the pair kernel and the finish kernel of every later call; None clears the hook."""
    handle = None
    if event is not None:
        handle = getattr(event, "cuda_event", event)
    return _load().fsd_set_stage_event(handle)


def fsd_debug_checks(B: int = 0, positions: int = 0):
    """(enabled, byte offset of the debug word in a workspace for this shape or None)."""
    off = C.c_size_t(0)
    on = _load().fsd_debug_checks(int(B), int(positions), C.byref(off))
    return bool(on), (off.value if B >= 1 and positions >= 1 else None)


def fsd_set_timeout_injection(mode) -> int:
    """Test aid.  1 (or True): verify calls report FSD_ROW_TIMEOUT in every row as if a bounded
    device-side wait had run out.  2: one thread block of the streaming kernel withholds a message,
    so that a (shortened) device-side wait really runs out.  0 (or False): off."""
    return _load().fsd_set_timeout_injection(int(mode))


def fsd_set_group_size(group_size: int) -> int:
    """Thread blocks a pair is split over in the streaming kernel (a test and tuning aid); 0: the
    library chooses."""
    return _load().fsd_set_group_size(int(group_size))


def fsd_workspace_bytes(B: int, positions: int, V: int, opts: FsdOpts) -> int:
    out = C.c_size_t(0)
    rc = _load().fsd_workspace_bytes(B, positions, V, C.byref(opts), C.byref(out))
    if rc != FSD_OK:
        raise FsdError(rc)
    return out.value


def fsd_verify_chain(target_logits, draft_logits, draft_tokens, u_accept, u_sample, B, gamma, V, opts,
                     accept_len, next_token, divergence, row_status, workspace, workspace_bytes, stream=None) -> int:
    """Same arguments as the C entry point; tensors (or integer addresses) are passed as pointers.
    Returns the host status code (0 = OK)."""
    return _load().fsd_verify_chain(_ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens), _ptr(u_accept),
                                    _ptr(u_sample), B, gamma, V, C.byref(opts) if opts is not None else None,
                                    _ptr(accept_len), _ptr(next_token), _ptr(divergence), _ptr(row_status),
                                    _ptr(workspace), int(workspace_bytes), _ptr(stream))


def fsd_verify_tree(target_logits, draft_logits, parent, u_sample, B, N, V, max_depth, opts,
                    accept_len, path, next_token, divergence, row_status, workspace, workspace_bytes,
                    stream=None) -> int:
    return _load().fsd_verify_tree(_ptr(target_logits), _ptr(draft_logits), _ptr(parent), _ptr(u_sample),
                                   B, N, V, max_depth, C.byref(opts) if opts is not None else None,
                                   _ptr(accept_len), _ptr(path), _ptr(next_token), _ptr(divergence),
                                   _ptr(row_status), _ptr(workspace), int(workspace_bytes), _ptr(stream))


def fsd_host_staging_bytes(B: int, gamma: int, V: int, opts: FsdOpts) -> int:
    out = C.c_size_t(0)
    rc = _load().fsd_host_staging_bytes(B, gamma, V, C.byref(opts), C.byref(out))
    if rc != FSD_OK:
        raise FsdError(rc)
    return out.value


def fsd_verify_chain_host(h_target_logits, h_draft_logits, h_draft_tokens, h_u_accept, h_u_sample, B, gamma, V,
                          opts, h_accept_len, h_next_token, h_divergence, h_row_status, staging, staging_bytes,
                          stream=None) -> int:
    """Host-buffer variant: the h_* arguments are CPU tensors (ideally pinned), `staging` a device tensor."""
    return _load().fsd_verify_chain_host(_ptr(h_target_logits), _ptr(h_draft_logits), _ptr(h_draft_tokens),
                                         _ptr(h_u_accept), _ptr(h_u_sample), B, gamma, V,
                                         C.byref(opts) if opts is not None else None, _ptr(h_accept_len),
                                         _ptr(h_next_token), _ptr(h_divergence), _ptr(h_row_status),
                                         _ptr(staging), int(staging_bytes), _ptr(stream))


def fsd_verify_chain_static(target_logits, draft_logits, draft_tokens, u_accept, u_sample, B, gamma, V, opts,
                            accept_len, next_token, divergence, row_status, stream=None) -> int:
    """fsd_verify_chain for callers that may not allocate device memory: no workspace argument,
    the scratch lives inside the library (B * gamma <= FSD_STATIC_MAX_POSITIONS)."""
    return _load().fsd_verify_chain_static(_ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens),
                                           _ptr(u_accept), _ptr(u_sample), B, gamma, V,
                                           C.byref(opts) if opts is not None else None, _ptr(accept_len),
                                           _ptr(next_token), _ptr(divergence), _ptr(row_status), _ptr(stream))



def fsd_threshold_sweep(divergence, B, positions, thresholds, n_thresholds, compare, mean_accept_len,
                        accept_fraction, stream=None) -> int:
    return _load().fsd_threshold_sweep(_ptr(divergence), B, positions, _ptr(thresholds), n_thresholds, compare,
                                       _ptr(mean_accept_len), _ptr(accept_fraction), stream)


def fsd_calibrate_threshold(divergence, B, positions, target_mean_accept_len, compare, threshold_out, achieved_out,
                            stream=None) -> int:
    return _load().fsd_calibrate_threshold(_ptr(divergence), B, positions, float(target_mean_accept_len), compare,
                                           _ptr(threshold_out), _ptr(achieved_out), stream)


def fsd_accept_labels(divergence, B, positions, threshold, compare, labels, stream=None) -> int:
    return _load().fsd_accept_labels(_ptr(divergence), B, positions, float(threshold), compare, _ptr(labels), stream)
