"""TEST INFRASTRUCTURE: ctypes front end of the plain CPU fp64 oracle (pp_oracle.c).

Only tests, the smoke check and the benchmark's cpu_baseline / reference legs may
import this package.  It shares no code with the CUDA library and never imports it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pp_oracle.c")
_LIB = os.path.join(_HERE, "libpp_oracle.so")
_lib: Optional[ctypes.CDLL] = None


class _Desc(ctypes.Structure):
    _fields_ = [("num_rows", ctypes.c_int32),
                ("row_group_off", ctypes.c_void_p),
                ("grp_prompt_len", ctypes.c_void_p),
                ("grp_resp_off", ctypes.c_void_p),
                ("resp_len", ctypes.c_void_p)]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP) into oracle/libpp_oracle.so."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.ppo_token_ids.restype = ctypes.c_long
    return _lib


def max_threads() -> int:
    return int(lib().ppo_max_threads())


def _desc(row_group_off, grp_prompt_len, grp_resp_off, resp_len):
    arrs = [np.ascontiguousarray(a, dtype=np.int32)
            for a in (row_group_off, grp_prompt_len, grp_resp_off, resp_len)]
    d = _Desc(len(arrs[0]) - 1, *[a.ctypes.data for a in arrs])
    return d, arrs


def _bits(x) -> np.ndarray:
    """bf16 torch tensor (or uint16 array) -> contiguous uint16 bit patterns."""
    if isinstance(x, np.ndarray):
        assert x.dtype == np.uint16
        return np.ascontiguousarray(x)
    import torch
    assert x.dtype == torch.bfloat16
    return np.ascontiguousarray(x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16))


def _p(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def token_ids(desc):
    d, keep = _desc(*desc)
    T = lib().ppo_token_ids(ctypes.byref(d), None, None, None)
    if T < 0:
        raise ValueError(f"oracle rejected descriptors ({T})")
    out = [np.empty(T, dtype=np.int32) for _ in range(3)]
    lib().ppo_token_ids(ctypes.byref(d), _p(out[0]), _p(out[1]), _p(out[2]))
    return tuple(out)


def dense_mask(desc, row: int) -> np.ndarray:
    d, keep = _desc(*desc)
    tr, _, _ = token_ids(desc)
    L = int((tr == row).sum())
    m = np.empty((L, L), dtype=np.uint8)
    rc = lib().ppo_dense_mask(ctypes.byref(d), ctypes.c_int(row), _p(m))
    if rc:
        raise ValueError(f"ppo_dense_mask failed ({rc})")
    return m.astype(bool)


def attn_fwd(desc, q, k, v, scale: float, num_threads: int = 0):
    """Returns (O [T,Hq,D] f64, LSE [Hq,T] f64)."""
    d, keep = _desc(*desc)
    qb, kb, vb = _bits(q), _bits(k), _bits(v)
    T, Hq, D = qb.shape
    Hkv = kb.shape[1]
    O = np.empty((T, Hq, D), dtype=np.float64)
    LSE = np.empty((Hq, T), dtype=np.float64)
    rc = lib().ppo_attn_fwd(ctypes.byref(d), Hq, Hkv, D, _p(qb), _p(kb), _p(vb),
                            ctypes.c_double(float(scale)), _p(O), _p(LSE), int(num_threads))
    if rc:
        raise ValueError(f"ppo_attn_fwd failed ({rc})")
    return O, LSE


def attn_fwd_bwd(desc, q, k, v, dout, scale: float, num_threads: int = 0):
    """Returns (O, LSE, dQ, dK, dV) in fp64."""
    d, keep = _desc(*desc)
    qb, kb, vb, dob = _bits(q), _bits(k), _bits(v), _bits(dout)
    T, Hq, D = qb.shape
    Hkv = kb.shape[1]
    O = np.empty((T, Hq, D), dtype=np.float64)
    LSE = np.empty((Hq, T), dtype=np.float64)
    dQ = np.empty((T, Hq, D), dtype=np.float64)
    dK = np.empty((T, Hkv, D), dtype=np.float64)
    dV = np.empty((T, Hkv, D), dtype=np.float64)
    rc = lib().ppo_attn_fwd_bwd(ctypes.byref(d), Hq, Hkv, D, _p(qb), _p(kb), _p(vb), _p(dob),
                                ctypes.c_double(float(scale)), _p(O), _p(LSE), _p(dQ), _p(dK),
                                _p(dV), int(num_threads))
    if rc:
        raise ValueError(f"ppo_attn_fwd_bwd failed ({rc})")
    return O, LSE, dQ, dK, dV


def dump_intermediates(desc, q, k, v, dout, scale: float, row: int, head: int):
    """Dense (S, P, dP, dS), each [L, L], of one (row, query head); tiny cases only."""
    d, keep = _desc(*desc)
    qb, kb, vb, dob = _bits(q), _bits(k), _bits(v), _bits(dout)
    T, Hq, D = qb.shape
    Hkv = kb.shape[1]
    tr, _, _ = token_ids(desc)
    L = int((tr == row).sum())
    out = [np.empty((L, L), dtype=np.float64) for _ in range(4)]
    rc = lib().ppo_dump_intermediates(ctypes.byref(d), Hq, Hkv, D, _p(qb), _p(kb), _p(vb), _p(dob),
                                      ctypes.c_double(float(scale)), row, head,
                                      *[_p(o) for o in out])
    if rc:
        raise ValueError(f"ppo_dump_intermediates failed ({rc})")
    return tuple(out)
