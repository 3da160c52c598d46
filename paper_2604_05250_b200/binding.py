"""Thin ctypes binding of ``include/dualdiff.h``: argument marshalling only.

Every function takes torch tensors (device memory for the plain calls, pinned
host memory for the ``*_host`` calls), passes their data pointers and sizes
through the C ABI, and raises ``DualDiffError`` on a non-zero status.  There is
no Python or CPU implementation behind these names: if ``libdualdiff.so`` is
missing the first call raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdualdiff.so")

DD_OK, DD_ERR_INVALID_ARG, DD_ERR_UNSUPPORTED, DD_ERR_CUDA, DD_ERR_TIMEOUT = 0, -1, -2, -3, -4
DD_MODE_TRUST, DD_MODE_KL, DD_MODE_CONF = 0, 1, 2
DD_FLAG_PROBABILISTIC, DD_FLAG_EMIT_DRAFTER = 0x100, 0x200
DD_LAYOUT_BHND, DD_LAYOUT_BNHD = 0, 1

# every symbol include/dualdiff.h declares
EXPORTS = (
    "dd_bidir_attention", "dd_block_attention", "dd_verify", "dd_unmask", "dd_bidir_attention_host", "dd_verify_host", "dd_verify_static",
    "dd_verify_workspace_bytes", "dd_attention_status", "dd_verify_status", "dd_launch_count", "dd_release",
    "dd_status_string", "dd_last_cuda_error", "dd_version", "dd_debug_set_max_ctas", "dd_clear_status", "dd_debug_expire_wait", "dd_lm_head_verify",
)


class DualDiffError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"dualdiff status {status}: {text}")
        self.status = status


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libdualdiff.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        _lib = load(LIB_PATH)
    return _lib


class use_library:
    """Context manager: the wrappers below call the library at `path` (for instance the
    bounds-checked build) instead of libdualdiff.so until the block ends."""

    def __init__(self, path):
        self.path = path

    def __enter__(self):
        global _lib
        self.saved = _lib
        _lib = load(self.path)
        return _lib

    def __exit__(self, *exc):
        global _lib
        _lib = self.saved
        return False


def load(path) -> ctypes.CDLL:
    """Loads one build of the library and declares its entry points."""
    if True:
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: build it with `python -m paper_2604_05250_b200.build`; "
                "there is no fallback implementation")
        L = ctypes.CDLL(path)
        vp, i32, f32, u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_uint64
        attn = [vp, vp, vp, vp, i32, i32, i32, i32, f32, vp]
        ver = [vp, vp, vp, vp, i32, f32, i32, u64, vp, vp, vp, i32, i32, i32, vp]
        L.dd_bidir_attention.argtypes = attn
        L.dd_bidir_attention_host.argtypes = attn
        L.dd_block_attention.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, i32, f32, vp]
        L.dd_block_attention.restype = i32
        L.dd_verify.argtypes = ver
        L.dd_verify_host.argtypes = ver
        L.dd_verify_static.argtypes = ver
        L.dd_unmask.argtypes = [vp, vp, vp, f32, i32, vp, vp, vp, i32, i32, i32, vp]
        L.dd_unmask.restype = i32
        L.dd_verify_static.restype = i32
        for name in ("dd_bidir_attention", "dd_bidir_attention_host", "dd_verify", "dd_verify_host",
                     "dd_attention_status", "dd_verify_status", "dd_release", "dd_version"):
            getattr(L, name).restype = i32
        L.dd_attention_status.argtypes = []
        L.dd_verify_status.argtypes = []
        L.dd_release.argtypes = []
        L.dd_version.argtypes = []
        L.dd_verify_workspace_bytes.argtypes = [i32, i32, i32]
        L.dd_verify_workspace_bytes.restype = ctypes.c_size_t
        L.dd_launch_count.argtypes = []
        L.dd_launch_count.restype = u64
        L.dd_lm_head_verify.argtypes = [vp, vp, vp, vp, vp, vp, i32, f32, i32, u64, vp, vp, vp, i32, i32, i32, i32, vp]
        L.dd_lm_head_verify.restype = i32
        L.dd_clear_status.argtypes = []
        L.dd_clear_status.restype = i32
        L.dd_debug_expire_wait.argtypes = [i32, vp]
        L.dd_debug_expire_wait.restype = i32
        L.dd_debug_set_max_ctas.argtypes = [i32]
        L.dd_debug_set_max_ctas.restype = i32
        L.dd_status_string.argtypes = [i32]
        L.dd_status_string.restype = ctypes.c_char_p
        L.dd_last_cuda_error.argtypes = []
        L.dd_last_cuda_error.restype = ctypes.c_char_p
    return L


def _check(status: int):
    if status != DD_OK:
        L = lib()
        text = L.dd_status_string(status).decode()
        if status == DD_ERR_CUDA:
            text += ": " + L.dd_last_cuda_error().decode()
        raise DualDiffError(status, text)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _require(t, dtype, shape, cuda, name):
    import torch
    if not isinstance(t, torch.Tensor):
        raise TypeError(f"{name}: expected a torch.Tensor")
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise ValueError(f"{name}: expected contiguous {dtype} of shape {tuple(shape)}, "
                         f"got {t.dtype} {tuple(t.shape)}")
    if t.is_cuda != cuda:
        raise ValueError(f"{name}: expected a {'device' if cuda else 'host'} tensor")


def bidir_attention(q, k, v, out=None, scale=None, stream=None, host=False):
    """dd_bidir_attention (dd_bidir_attention_host if host=True).

    q, k, v: [B,H,N,D] torch.bfloat16.  Returns out (allocated if None)."""
    import torch
    B, H, N, D = q.shape
    cuda = not host
    for name, t in (("q", q), ("k", k), ("v", v)):
        _require(t, torch.bfloat16, (B, H, N, D), cuda, name)
    if out is None:
        out = torch.empty_like(q)
    _require(out, torch.bfloat16, (B, H, N, D), cuda, "out")
    if scale is None:
        scale = float(D) ** -0.5
    fn = lib().dd_bidir_attention_host if host else lib().dd_bidir_attention
    _check(fn(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, N, D, float(scale), _stream_ptr(stream)))
    return out


def block_attention(q, k, v, kv_len=None, layout="bhnd", out=None, scale=None, stream=None):
    """dd_block_attention: a block of Nq queries over Nkv stored keys and values.

    layout "bhnd": q [B,H,Nq,D], k, v [B,H,Nkv,D]; "bnhd": q [B,Nq,H,D], k, v [B,Nkv,H,D];
    torch.bfloat16 device tensors.  kv_len: int32 [B] device tensor (valid keys per sequence)
    or None.  Returns out (allocated if None), in the layout of q."""
    import torch
    if layout == "bhnd":
        B, H, Nq, D = q.shape
        Nkv = k.shape[2]
        kshape = (B, H, Nkv, D)
    elif layout == "bnhd":
        B, Nq, H, D = q.shape
        Nkv = k.shape[1]
        kshape = (B, Nkv, H, D)
    else:
        raise ValueError("layout: 'bhnd' or 'bnhd'")
    _require(q, torch.bfloat16, tuple(q.shape), True, "q")
    _require(k, torch.bfloat16, kshape, True, "k")
    _require(v, torch.bfloat16, kshape, True, "v")
    if kv_len is not None:
        _require(kv_len, torch.int32, (B,), True, "kv_len")
    if out is None:
        out = torch.empty_like(q)
    _require(out, torch.bfloat16, tuple(q.shape), True, "out")
    if scale is None:
        scale = float(D) ** -0.5
    _check(lib().dd_block_attention(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, Nq, Nkv, D, _ptr(kv_len),
                                    DD_LAYOUT_BHND if layout == "bhnd" else DD_LAYOUT_BNHD, float(scale),
                                    _stream_ptr(stream)))
    return out


def verify(drafter_logits, verifier_logits, tokens, mask_flags, mode, tau, k, seed,
           out_tokens=None, out_mask=None, out_score=None, want_score=True, stream=None, host=False,
           static_scratch=False):
    """dd_verify (dd_verify_host if host=True; dd_verify_static, the variant that allocates
    nothing, if static_scratch=True and every output tensor is passed in).

    Returns (out_tokens int32 [B,P], out_mask uint8 [B,P], out_score float32 [B,P] or None)."""
    import torch
    B, P, V = verifier_logits.shape
    cuda = not host
    _require(verifier_logits, torch.bfloat16, (B, P, V), cuda, "verifier_logits")
    if drafter_logits is not None:
        _require(drafter_logits, torch.bfloat16, (B, P, V), cuda, "drafter_logits")
    _require(tokens, torch.int32, (B, P), cuda, "tokens")
    _require(mask_flags, torch.uint8, (B, P), cuda, "mask_flags")
    kw = dict(device=verifier_logits.device, pin_memory=host)
    if out_tokens is None:
        out_tokens = torch.empty((B, P), dtype=torch.int32, **kw)
    if out_mask is None:
        out_mask = torch.empty((B, P), dtype=torch.uint8, **kw)
    if out_score is None and want_score:
        out_score = torch.empty((B, P), dtype=torch.float32, **kw)
    _require(out_tokens, torch.int32, (B, P), cuda, "out_tokens")
    _require(out_mask, torch.uint8, (B, P), cuda, "out_mask")
    if out_score is not None:
        _require(out_score, torch.float32, (B, P), cuda, "out_score")
    fn = lib().dd_verify_host if host else (lib().dd_verify_static if static_scratch else lib().dd_verify)
    _check(fn(_ptr(drafter_logits), _ptr(verifier_logits), _ptr(tokens), _ptr(mask_flags),
              int(mode), float(tau), int(k), int(seed) & 0xFFFFFFFFFFFFFFFF,
              _ptr(out_tokens), _ptr(out_mask), _ptr(out_score), B, P, V, _stream_ptr(stream)))
    return out_tokens, out_mask, out_score


def lm_head_verify(drafter_hidden, drafter_weight, verifier_hidden, verifier_weight, tokens, mask_flags,
                   mode, tau, k, seed, out_tokens=None, out_mask=None, out_score=None, stream=None):
    """dd_lm_head_verify: the language-model heads fused with the verification algorithm.

    verifier_hidden [B,P,K], verifier_weight [V,K]: torch.bfloat16 device tensors; drafter_hidden,
    drafter_weight: the same shapes, or None in the modes that need the verifier only.
    Returns (out_tokens int32 [B,P], out_mask uint8 [B,P], out_score float32 [B,P])."""
    import torch
    B, P, K = verifier_hidden.shape
    V = verifier_weight.shape[0]
    if drafter_hidden is not None:
        _require(drafter_hidden, torch.bfloat16, (B, P, K), True, "drafter_hidden")
    if drafter_weight is not None:
        _require(drafter_weight, torch.bfloat16, (V, K), True, "drafter_weight")
    _require(verifier_hidden, torch.bfloat16, (B, P, K), True, "verifier_hidden")
    _require(verifier_weight, torch.bfloat16, (V, K), True, "verifier_weight")
    _require(tokens, torch.int32, (B, P), True, "tokens")
    _require(mask_flags, torch.uint8, (B, P), True, "mask_flags")
    kw = dict(device=verifier_hidden.device)
    if out_tokens is None:
        out_tokens = torch.empty((B, P), dtype=torch.int32, **kw)
    if out_mask is None:
        out_mask = torch.empty((B, P), dtype=torch.uint8, **kw)
    if out_score is None:
        out_score = torch.empty((B, P), dtype=torch.float32, **kw)
    _require(out_tokens, torch.int32, (B, P), True, "out_tokens")
    _require(out_mask, torch.uint8, (B, P), True, "out_mask")
    _require(out_score, torch.float32, (B, P), True, "out_score")
    _check(lib().dd_lm_head_verify(_ptr(drafter_hidden), _ptr(drafter_weight), _ptr(verifier_hidden),
                                   _ptr(verifier_weight), _ptr(tokens), _ptr(mask_flags),
                                   int(mode), float(tau), int(k), int(seed) & 0xFFFFFFFFFFFFFFFF,
                                   _ptr(out_tokens), _ptr(out_mask), _ptr(out_score), B, P, K, V, _stream_ptr(stream)))
    return out_tokens, out_mask, out_score


def unmask(logits, tokens, mask_flags, tau, k, out_tokens=None, out_mask=None, out_conf=None, stream=None):
    """dd_unmask: one confidence-based unmasking step on logits [B,P,V] (device tensors).

    Returns (out_tokens int32 [B,P], out_mask uint8 [B,P] with 1 = still masked, out_conf float32 [B,P])."""
    import torch
    B, P, V = logits.shape
    _require(logits, torch.bfloat16, (B, P, V), True, "logits")
    _require(tokens, torch.int32, (B, P), True, "tokens")
    _require(mask_flags, torch.uint8, (B, P), True, "mask_flags")
    kw = dict(device=logits.device)
    if out_tokens is None:
        out_tokens = torch.empty((B, P), dtype=torch.int32, **kw)
    if out_mask is None:
        out_mask = torch.empty((B, P), dtype=torch.uint8, **kw)
    if out_conf is None:
        out_conf = torch.empty((B, P), dtype=torch.float32, **kw)
    _require(out_tokens, torch.int32, (B, P), True, "out_tokens")
    _require(out_mask, torch.uint8, (B, P), True, "out_mask")
    _require(out_conf, torch.float32, (B, P), True, "out_conf")
    _check(lib().dd_unmask(_ptr(logits), _ptr(tokens), _ptr(mask_flags), float(tau), int(k),
                           _ptr(out_tokens), _ptr(out_mask), _ptr(out_conf), B, P, V, _stream_ptr(stream)))
    return out_tokens, out_mask, out_conf


def attention_status() -> int:
    return int(lib().dd_attention_status())


def verify_status() -> int:
    return int(lib().dd_verify_status())


def launch_count() -> int:
    return int(lib().dd_launch_count())


def debug_set_max_ctas(n: int):
    """Test hook: cap the grid of the streaming verify kernel (0 = no cap)."""
    _check(lib().dd_debug_set_max_ctas(int(n)))


def clear_status():
    """Re-arms the kernels' health words on the current device after a recorded timeout."""
    _check(lib().dd_clear_status())


def debug_expire_wait(which: int, stream=None):
    """Test hook: records an expired wait for the attention kernel (0) or dd_verify (1)."""
    _check(lib().dd_debug_expire_wait(int(which), _stream_ptr(stream)))


def release():
    _check(lib().dd_release())


def version() -> int:
    return int(lib().dd_version())


def verify_workspace_bytes(B, P, V) -> int:
    return int(lib().dd_verify_workspace_bytes(B, P, V))
