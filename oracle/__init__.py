"""CPU oracle for one DualDiffusion verification step -- TEST INFRASTRUCTURE ONLY.

A ctypes loader around ``dd_oracle.c`` (plain fp64 C).  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may import this package; the
CUDA library never does, and this package imports nothing from it.

Arrays cross the boundary as numpy arrays: bf16 tensors as ``uint16`` bit
patterns, everything else in its natural dtype.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dd_oracle.c")
_LIB = os.path.join(_HERE, "libdd_oracle.so")

MODE_TRUST, MODE_KL, MODE_CONF = 0, 1, 2
FLAG_PROBABILISTIC, FLAG_EMIT_DRAFTER = 0x100, 0x200

_lib = None


def build(force: bool = False) -> str:
    """Compile dd_oracle.c into libdd_oracle.so with gcc (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        vp, i32, f64, u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_uint64
        lib.dd_oracle_attention.argtypes = [vp, vp, vp, i32, i32, i32, i32, f64, vp, i32, vp, vp]
        lib.dd_oracle_attention.restype = None
        lib.dd_oracle_attention_probs.argtypes = [vp, vp, i32, i32, i32, f64, i32, i32, i32, vp]
        lib.dd_oracle_attention_probs.restype = None
        lib.dd_oracle_block_attention.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, i32, f64, vp]
        lib.dd_oracle_block_attention.restype = None
        lib.dd_oracle_philox4x32_10.argtypes = [vp, vp, vp]
        lib.dd_oracle_philox4x32_10.restype = None
        lib.dd_oracle_uniform.argtypes = [u64, i32, i32]
        lib.dd_oracle_uniform.restype = f64
        lib.dd_oracle_row_scores.argtypes = [vp, vp, i32, vp, vp, vp]
        lib.dd_oracle_row_scores.restype = None
        lib.dd_oracle_verify.argtypes = [vp, vp, vp, vp, i32, f64, i32, u64,
                                         vp, vp, vp, vp, i32, i32, i32]
        lib.dd_oracle_verify.restype = i32
        lib.dd_oracle_verify_f64.argtypes = [vp, vp, vp, vp, i32, f64, i32, u64,
                                             vp, vp, vp, vp, i32, i32, i32]
        lib.dd_oracle_verify_f64.restype = i32
        lib.dd_oracle_lm_head.argtypes = [vp, vp, vp, i32, i32, i32, vp]
        lib.dd_oracle_lm_head.restype = None
        lib.dd_oracle_unmask.argtypes = [vp, vp, vp, f64, i32, vp, vp, vp, vp, i32, i32, i32]
        lib.dd_oracle_unmask.restype = None
        lib.dd_oracle_threads.argtypes = []
        lib.dd_oracle_threads.restype = i32
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a, shape=None):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 tensors are passed as uint16 bit patterns"
    if shape is not None:
        assert a.shape == tuple(shape), (a.shape, shape)
    return a


def threads() -> int:
    return int(_load().dd_oracle_threads())


def attention(q, k, v, scale, rows=None, return_lse=False):
    """Eq. 3 over the whole key range.  q,k,v: [B,H,N,D] uint16 (bf16 bits).

    Returns out [B,H,R,D] float64 (R = len(rows) or N), optionally the row LSE.
    """
    q = _u16(q)
    B, H, N, D = q.shape
    k = _u16(k, q.shape)
    v = _u16(v, q.shape)
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int32)
        assert rows.ndim == 1 and rows.size > 0 and rows.min() >= 0 and rows.max() < N
    R = N if rows is None else rows.size
    out = np.empty((B, H, R, D), dtype=np.float64)
    lse = np.empty((B, H, R), dtype=np.float64)
    _load().dd_oracle_attention(_ptr(q), _ptr(k), _ptr(v), B, H, N, D, float(scale),
                                _ptr(rows), 0 if rows is None else rows.size,
                                _ptr(out), _ptr(lse))
    return (out, lse) if return_lse else out


def block_attention(q, k, v, scale, kv_len=None, layout="bhnd"):
    """Eq. 3 for a block of queries over stored keys (Section 2.3's cached drafter step).

    layout "bhnd": q [B,H,Nq,D], k,v [B,H,Nkv,D]; "bnhd": q [B,Nq,H,D], k,v [B,Nkv,H,D]
    (uint16 bf16 bits).  kv_len: int32 [B] valid keys per sequence, or None.
    Returns float64 in the layout of q."""
    assert layout in ("bhnd", "bnhd")
    q = _u16(q)
    k = _u16(k)
    if layout == "bhnd":
        B, H, Nq, D = q.shape
        Nkv = k.shape[2]
        assert k.shape == (B, H, Nkv, D)
    else:
        B, Nq, H, D = q.shape
        Nkv = k.shape[1]
        assert k.shape == (B, Nkv, H, D)
    v = _u16(v, k.shape)
    if kv_len is not None:
        kv_len = np.ascontiguousarray(kv_len, dtype=np.int32)
        assert kv_len.shape == (B,)
    out = np.empty(q.shape, dtype=np.float64)
    _load().dd_oracle_block_attention(_ptr(q), _ptr(k), _ptr(v), B, H, Nq, Nkv, D, _ptr(kv_len),
                                      1 if layout == "bhnd" else 0, float(scale), _ptr(out))
    return out


def attention_probs(q, k, scale, b, h, i):
    """Softmax weights of query row i of head (b,h): float64 [N]."""
    q = _u16(q)
    B, H, N, D = q.shape
    k = _u16(k, q.shape)
    p = np.empty(N, dtype=np.float64)
    _load().dd_oracle_attention_probs(_ptr(q), _ptr(k), H, N, D, float(scale), b, h, i, _ptr(p))
    return p


def philox4x32_10(counter, key):
    c = np.ascontiguousarray(counter, dtype=np.uint32)
    kk = np.ascontiguousarray(key, dtype=np.uint32)
    assert c.shape == (4,) and kk.shape == (2,)
    out = np.empty(4, dtype=np.uint32)
    _load().dd_oracle_philox4x32_10(_ptr(c), _ptr(kk), _ptr(out))
    return out


def uniform(seed, b, i) -> float:
    return float(_load().dd_oracle_uniform(int(seed), int(b), int(i)))


def row_scores(drafter_row, verifier_row):
    """(argmax_v, c_V, KL(p_D||p_V)) for one position; drafter_row may be None."""
    vr = _u16(verifier_row)
    dr = None if drafter_row is None else _u16(drafter_row, vr.shape)
    a = ctypes.c_int32(0)
    c = ctypes.c_double(0.0)
    kl = ctypes.c_double(0.0)
    _load().dd_oracle_row_scores(_ptr(dr), _ptr(vr), vr.size,
                                 ctypes.byref(a), ctypes.byref(c), ctypes.byref(kl))
    return int(a.value), float(c.value), float(kl.value)


def verify(drafter, verifier, tokens, flags, mode, tau, k, seed):
    """Verification algorithm A of Algorithm 1.  Returns a dict with
    out_tokens int32 [B,P], out_mask uint8 [B,P], out_score float64 [B,P],
    exempt uint8 [B,P]."""
    verifier = _u16(verifier)
    B, P, V = verifier.shape
    drafter = None if drafter is None else _u16(drafter, verifier.shape)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    flags = np.ascontiguousarray(flags, dtype=np.uint8)
    assert tokens.shape == (B, P) and flags.shape == (B, P)
    out_tokens = np.empty((B, P), dtype=np.int32)
    out_mask = np.empty((B, P), dtype=np.uint8)
    out_score = np.empty((B, P), dtype=np.float64)
    exempt = np.empty((B, P), dtype=np.uint8)
    # tau reaches the CUDA library as a C float: the oracle compares against the same value
    tau32 = float(np.float32(tau))
    rc = _load().dd_oracle_verify(_ptr(drafter), _ptr(verifier), _ptr(tokens), _ptr(flags),
                                  int(mode), tau32, int(k), int(seed),
                                  _ptr(out_tokens), _ptr(out_mask), _ptr(out_score),
                                  _ptr(exempt), B, P, V)
    if rc != 0:
        raise ValueError(f"dd_oracle_verify rejected its arguments (rc={rc})")
    return dict(out_tokens=out_tokens, out_mask=out_mask, out_score=out_score, exempt=exempt)


def lm_head(hidden, weight, flags=None):
    """Logits of the language-model head: hidden [rows,K] x weight [V,K]^T in fp64 (uint16 bf16 bits in).
    Rows with flag 0 are skipped (zeros).  Returns float64 [rows,V]."""
    hidden, weight = _u16(hidden), _u16(weight)
    rows, K = hidden.shape
    V = weight.shape[0]
    assert weight.shape == (V, K)
    if flags is not None:
        flags = np.ascontiguousarray(flags, dtype=np.uint8).reshape(rows)
    out = np.empty((rows, V), dtype=np.float64)
    _load().dd_oracle_lm_head(_ptr(hidden), _ptr(weight), _ptr(flags), rows, K, V, _ptr(out))
    return out


def verify_f64(drafter, verifier, tokens, flags, mode, tau, k, seed):
    """Verification algorithm A on fp64 logits [B,P,V] (what a fused language-model head hands over
    without rounding).  Same outputs as verify()."""
    verifier = np.ascontiguousarray(verifier, dtype=np.float64)
    B, P, V = verifier.shape
    if drafter is not None:
        drafter = np.ascontiguousarray(drafter, dtype=np.float64)
        assert drafter.shape == verifier.shape
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    flags = np.ascontiguousarray(flags, dtype=np.uint8)
    assert tokens.shape == (B, P) and flags.shape == (B, P)
    out_tokens = np.empty((B, P), dtype=np.int32)
    out_mask = np.empty((B, P), dtype=np.uint8)
    out_score = np.empty((B, P), dtype=np.float64)
    exempt = np.empty((B, P), dtype=np.uint8)
    rc = _load().dd_oracle_verify_f64(_ptr(drafter), _ptr(verifier), _ptr(tokens), _ptr(flags),
                                      int(mode), float(np.float32(tau)), int(k), int(seed),
                                      _ptr(out_tokens), _ptr(out_mask), _ptr(out_score), _ptr(exempt), B, P, V)
    if rc != 0:
        raise ValueError(f"dd_oracle_verify_f64 rejected its arguments (rc={rc})")
    return dict(out_tokens=out_tokens, out_mask=out_mask, out_score=out_score, exempt=exempt)


def lm_head_verify(hidden_d, weight_d, hidden_v, weight_v, tokens, flags, mode, tau, k, seed, round_logits=False):
    """The verification phase from the models' last hidden states: logits by lm_head(), then the
    verification algorithm.  hidden_* [B,P,K], weight_* [V,K] (uint16 bf16 bits; the drafter pair may
    be None unless the mode is KL).  round_logits: round the logits to bf16 first (what an unfused
    head stores) and run verify() on them; otherwise verify_f64() on the fp64 logits.
    Adds `top2_gap` [B,P]: difference of the two largest verifier logits (token ids are only
    comparable where it exceeds what fp32 accumulation can blur)."""
    B, P, K = hidden_v.shape
    fl = np.ascontiguousarray(flags, dtype=np.uint8)
    lv = lm_head(np.ascontiguousarray(hidden_v).reshape(B * P, K), weight_v, fl)
    ld = None
    if hidden_d is not None:
        ld = lm_head(np.ascontiguousarray(hidden_d).reshape(B * P, K), weight_d, fl)
    V = lv.shape[1]
    part = np.partition(lv, V - 2, axis=1)
    gap = (part[:, V - 1] - part[:, V - 2]).reshape(B, P)
    if round_logits:
        to_bits = lambda a: ((a.astype(np.float32).view(np.uint32) + (((a.astype(np.float32).view(np.uint32) >> 16) & 1) + 0x7FFF)) >> 16).astype(np.uint16)
        r = verify(None if ld is None else to_bits(ld).reshape(B, P, V), to_bits(lv).reshape(B, P, V),
                   tokens, flags, mode, tau, k, seed)
    else:
        r = verify_f64(None if ld is None else ld.reshape(B, P, V), lv.reshape(B, P, V), tokens, flags, mode, tau, k, seed)
    r["top2_gap"] = gap
    return r


def unmask(logits, tokens, flags, tau, k):
    """One confidence-based unmasking step (Algorithm 1's Unmask).  Returns a dict with
    out_tokens int32 [B,P], out_mask uint8 [B,P] (1 = still masked), out_conf float64 [B,P],
    exempt uint8 [B,P]."""
    logits = _u16(logits)
    B, P, V = logits.shape
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    flags = np.ascontiguousarray(flags, dtype=np.uint8)
    assert tokens.shape == (B, P) and flags.shape == (B, P)
    out_tokens = np.empty((B, P), dtype=np.int32)
    out_mask = np.empty((B, P), dtype=np.uint8)
    out_conf = np.empty((B, P), dtype=np.float64)
    exempt = np.empty((B, P), dtype=np.uint8)
    tau32 = float(np.float32(tau))        # the CUDA library receives tau as a C float
    _load().dd_oracle_unmask(_ptr(logits), _ptr(tokens), _ptr(flags), tau32, int(k),
                             _ptr(out_tokens), _ptr(out_mask), _ptr(out_conf), _ptr(exempt), B, P, V)
    return dict(out_tokens=out_tokens, out_mask=out_mask, out_conf=out_conf, exempt=exempt)


def dualdiffusion_loop(drafter, verifier, tokens, mask_id, K, mode, tau, k, seed=0,
                       unmask_tau=float("inf"), unmask_k=1, max_cycles=10_000):
    """Algorithm 1 with the oracle's own Unmask and verification steps (numpy arrays throughout).

    drafter, verifier: callables tokens int32 [B,P] -> logits uint16 [B,P,V] (bf16 bits).
    Returns (tokens, dict of counters, number of decisions the oracle flagged as lying within
    its exemption band)."""
    x = np.array(tokens, dtype=np.int32, copy=True)
    stats = dict(cycles=0, drafter_calls=0, verifier_calls=0, unmasked_by_drafter=0,
                 remasked_by_verifier=0, masked_after_cycle=[])
    near = 0
    while stats["cycles"] < max_cycles:
        masked = x == mask_id
        if not masked.any():
            break
        drafted = np.zeros_like(masked)
        for _ in range(K):                                   # drafting phase
            if not masked.any():
                break
            r = unmask(drafter(x), x, masked.astype(np.uint8), unmask_tau, unmask_k)
            stats["drafter_calls"] += 1
            still = r["out_mask"].astype(bool)
            newly = masked & ~still
            drafted |= newly
            stats["unmasked_by_drafter"] += int(newly.sum())
            near += int(r["exempt"].sum())
            x = r["out_tokens"]
            masked = still
        logits_v = verifier(x)                               # verification phase
        stats["verifier_calls"] += 1
        logits_d = None
        if (mode & 0xFF) == 1:
            logits_d = drafter(x)
            stats["drafter_calls"] += 1
        r = verify(logits_d, logits_v, x, drafted.astype(np.uint8), mode, tau, k, seed + stats["cycles"])
        near += int(r["exempt"].sum())
        remask = r["out_mask"].astype(bool)
        x = np.where(remask, np.int32(mask_id), r["out_tokens"]).astype(np.int32)
        stats["remasked_by_verifier"] += int(remask.sum())
        stats["cycles"] += 1
        stats["masked_after_cycle"].append(int((x == mask_id).sum()))
    return x, stats, near
