"""Thin ctypes binding of libpp_attn.so: argument marshalling only.

Every step of the path (plan building, forward, backward) runs in the library's CUDA
kernels; PyTorch only provides device memory and the current stream.  There is no CPU
fallback: if the library is missing or no CUDA device is present, calls raise.

Function names mirror the C ABI (include/pp_attn.h): pp_build_plan, pp_attn_fwd,
pp_attn_bwd.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpp_attn.so")
_lib: Optional[ctypes.CDLL] = None

EXPORTS = ["pp_plan_workspace_bytes", "pp_build_plan", "pp_plan_status", "pp_destroy_plan",
           "pp_plan_max_tiles", "pp_plan_read", "pp_attn_fwd", "pp_attn_bwd",
           "pp_last_launch_count", "pp_error_string", "pp_step_host_arena_bytes", "pp_step_host_runs",
           "pp_attn_step_host", "pp_profile_enable", "pp_profile_read", "pp_profile_read_all",
           "pp_attn_bwd_noalloc", "pp_attn_bwd_noalloc_max_bytes", "pp_plan_read_bwd_units",
           "pp_plan_read_bwd_tiles", "pp_attn_bwd_deterministic",
           "pp_position_ids", "pp_rope_qk", "pp_preference_loss",
           "pp_build_rows_workspace_bytes", "pp_build_rows", "pp_assign_rows",
           "pp_debug_expire_wait"]


class PPError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().pp_error_string(code).decode()
        super().__init__(f"{where}: {msg} ({code})")


class _Problem(ctypes.Structure):
    _fields_ = [("num_rows", ctypes.c_int32),
                ("row_group_off", ctypes.c_void_p),
                ("grp_prompt_len", ctypes.c_void_p),
                ("grp_resp_off", ctypes.c_void_p),
                ("resp_len", ctypes.c_void_p),
                ("num_groups", ctypes.c_int32),
                ("num_responses", ctypes.c_int32),
                ("desc_on_device", ctypes.c_int32),
                ("num_q_heads", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32),
                ("total_tokens", ctypes.c_int32)]


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2602_24082_b200.build` (there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        L.pp_error_string.restype = ctypes.c_char_p
        L.pp_error_string.argtypes = [ctypes.c_int]
        vp, sz = ctypes.c_void_p, ctypes.c_size_t
        L.pp_plan_workspace_bytes.argtypes = [vp, vp, vp, vp]
        L.pp_build_plan.argtypes = [vp, vp, sz, vp, vp]
        L.pp_plan_status.argtypes = [vp, vp, vp, vp]
        L.pp_destroy_plan.argtypes = [vp]
        L.pp_plan_max_tiles.argtypes = [vp]
        L.pp_plan_read_bwd_units.argtypes = [vp, vp, vp]
        L.pp_plan_read_bwd_tiles.argtypes = [vp, vp, vp, vp]
        L.pp_plan_read.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.pp_attn_fwd.argtypes = [vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, sz, vp]
        L.pp_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, sz, vp]
        L.pp_attn_bwd_deterministic.argtypes = L.pp_attn_bwd.argtypes
        L.pp_build_rows_workspace_bytes.argtypes = [ctypes.c_int32, vp]
        L.pp_build_rows.argtypes = [ctypes.c_int32, ctypes.c_int32, vp, vp, vp, ctypes.c_int32, vp, sz] + [vp] * 10
        L.pp_assign_rows.argtypes = [ctypes.c_int32, vp, ctypes.c_int32, vp, vp, vp, vp]
        L.pp_debug_expire_wait.argtypes = [vp, ctypes.c_int32, vp]
        L.pp_step_host_arena_bytes.argtypes = [vp, vp]
        L.pp_step_host_runs.argtypes = [vp, vp, vp, vp]
        L.pp_attn_step_host.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, vp, vp, sz, vp]
        L.pp_attn_bwd_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp]
        L.pp_attn_bwd_noalloc_max_bytes.argtypes = [vp]
        L.pp_position_ids.argtypes = [vp, vp, vp]
        L.pp_rope_qk.argtypes = [vp, vp, vp, ctypes.c_float, vp]
        L.pp_preference_loss.argtypes = [vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, vp]
        L.pp_profile_enable.argtypes = [ctypes.c_int]
        L.pp_profile_read.argtypes = [vp, vp]
        L.pp_profile_read_all.argtypes = [vp, vp, ctypes.c_int32, vp, vp]
        _lib = L
    return _lib


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(rc: int, where: str):
    if rc != 0:
        raise PPError(rc, where)


class Plan:
    """Owns the host handle, the device workspace and the backward scratch of one problem."""

    def __init__(self, handle: int, problem: _Problem, workspace: torch.Tensor, keep, sizes):
        self.handle = handle
        self.problem = problem
        self.workspace = workspace
        self._keep = keep
        self.plan_bytes, self.fwd_scratch_bytes, self.bwd_scratch_bytes = sizes
        self._bwd_scratch: Optional[torch.Tensor] = None

    @property
    def total_tokens(self) -> int:
        return self.problem.total_tokens

    def bwd_scratch(self) -> torch.Tensor:
        if self._bwd_scratch is None:
            self._bwd_scratch = torch.empty(self.bwd_scratch_bytes, dtype=torch.uint8,
                                            device=self.workspace.device)
        return self._bwd_scratch

    def status(self) -> Tuple[int, int]:
        st, det = ctypes.c_int32(0), ctypes.c_int32(0)
        lib().pp_plan_status(self.handle, _stream(), ctypes.byref(st), ctypes.byref(det))
        return st.value, det.value

    def read(self):
        """(tiles [n,8], fwd_order [n], bwd_order [n], key_end [T]) as numpy arrays."""
        mt = lib().pp_plan_max_tiles(self.handle)
        tiles = np.zeros((mt, 8), dtype=np.int32)
        fo = np.zeros(mt, dtype=np.int32)
        bo = np.zeros(mt, dtype=np.int32)
        ke = np.zeros(self.total_tokens, dtype=np.int32)
        n = ctypes.c_int32(0)
        _check(lib().pp_plan_read(self.handle, _stream(), ctypes.byref(n), tiles.ctypes.data,
                                  fo.ctypes.data, bo.ctypes.data, ke.ctypes.data), "pp_plan_read")
        return tiles[:n.value], fo[:n.value], bo[:n.value], ke

    def read_bwd_tiles(self) -> np.ndarray:
        """Backward key tiles [n, 8]: start, len, vis_end, dep_lo, grp_start, grp_end, work, npc."""
        mt = lib().pp_plan_max_tiles(self.handle)
        bt = np.zeros((mt, 8), dtype=np.int32)
        n = ctypes.c_int32(0)
        _check(lib().pp_plan_read_bwd_tiles(self.handle, _stream(), ctypes.byref(n), bt.ctypes.data),
               "pp_plan_read_bwd_tiles")
        return bt[:n.value]

    def read_bwd_units(self, num_tiles: int) -> np.ndarray:
        """The backward processing order as (kv_head, backward tile) rows."""
        mt = lib().pp_plan_max_tiles(self.handle)
        hkv = self.problem.num_kv_heads
        raw = np.zeros(mt * hkv, dtype=np.int32)
        _check(lib().pp_plan_read_bwd_units(self.handle, _stream(), raw.ctypes.data),
               "pp_plan_read_bwd_units")
        raw = raw[:num_tiles * hkv]
        return np.stack([raw >> 24, raw & 0xffffff], axis=1)

    def __del__(self):
        try:
            if self.handle:
                lib().pp_destroy_plan(self.handle)
                self.handle = 0
        except Exception:
            pass


def make_problem(desc: Sequence[np.ndarray], num_q_heads: int, num_kv_heads: int, head_dim: int,
                 total_tokens: int, device_arrays: Optional[Sequence[torch.Tensor]] = None):
    """Fills a pp_problem.  ``desc`` = (row_group_off, grp_prompt_len, grp_resp_off, resp_len)."""
    arrs = [np.ascontiguousarray(a, dtype=np.int32) for a in desc]
    p = _Problem()
    p.num_rows = len(arrs[0]) - 1
    p.num_groups = len(arrs[1])
    p.num_responses = len(arrs[3])
    if device_arrays is not None:
        ptrs = [t.data_ptr() for t in device_arrays]
        p.desc_on_device = 1
    else:
        ptrs = [a.ctypes.data for a in arrs]
        p.desc_on_device = 0
    p.row_group_off, p.grp_prompt_len, p.grp_resp_off, p.resp_len = ptrs
    p.num_q_heads, p.num_kv_heads, p.head_dim = num_q_heads, num_kv_heads, head_dim
    p.total_tokens = total_tokens
    return p, (arrs, device_arrays)


def pp_plan_workspace_bytes(problem: _Problem) -> Tuple[int, int, int]:
    a, b, c = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib().pp_plan_workspace_bytes(ctypes.byref(problem), ctypes.byref(a), ctypes.byref(b),
                                         ctypes.byref(c)), "pp_plan_workspace_bytes")
    return a.value, b.value, c.value


def pp_build_plan(desc: Sequence[np.ndarray], num_q_heads: int, num_kv_heads: int, head_dim: int,
                  total_tokens: int, device: str = "cuda:0", desc_on_device: bool = False,
                  device_arrays: Optional[Sequence[torch.Tensor]] = None,
                  workspace: Optional[torch.Tensor] = None) -> Plan:
    """Builds a plan.  ``device_arrays`` (int32 CUDA tensors) and ``workspace`` (uint8 CUDA
    tensor of at least the queried size) let a caller re-plan every step without allocating."""
    if not torch.cuda.is_available():
        raise RuntimeError("pp_build_plan needs a CUDA device (there is no CPU fallback)")
    dev_arrays = device_arrays
    if desc_on_device and dev_arrays is None:
        dev_arrays = [torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device) for a in desc]
    problem, keep = make_problem(desc, num_q_heads, num_kv_heads, head_dim, total_tokens, dev_arrays)
    sizes = pp_plan_workspace_bytes(problem)
    ws = workspace if workspace is not None else torch.empty(sizes[0], dtype=torch.uint8, device=device)
    if ws.numel() < sizes[0]:
        raise ValueError("workspace too small")
    handle = ctypes.c_void_p(0)
    with torch.cuda.device(ws.device):
        _check(lib().pp_build_plan(ctypes.byref(problem), ws.data_ptr(), sizes[0], _stream(),
                                   ctypes.byref(handle)), "pp_build_plan")
    return Plan(handle.value, problem, ws, keep, sizes)


def _chk(t: torch.Tensor, shape, dtype, name):
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous() or not t.is_cuda:
        raise ValueError(f"{name}: expected contiguous CUDA {dtype} {tuple(shape)}, got "
                         f"{t.dtype} {tuple(t.shape)} on {t.device}")


def pp_attn_fwd(plan: Plan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                softmax_scale: float, o: Optional[torch.Tensor] = None,
                lse: Optional[torch.Tensor] = None, for_backward: bool = False):
    """``for_backward``: also hand the plan's backward scratch to the forward, which then clears
    the fp32 dQ accumulator in it (the following ``pp_attn_bwd`` skips its own clearing)."""
    p = plan.problem
    T, Hq, Hkv, D = p.total_tokens, p.num_q_heads, p.num_kv_heads, p.head_dim
    _chk(q, (T, Hq, D), torch.bfloat16, "q")
    _chk(k, (T, Hkv, D), torch.bfloat16, "k")
    _chk(v, (T, Hkv, D), torch.bfloat16, "v")
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty(Hq, T, dtype=torch.float32, device=q.device)
    _chk(o, (T, Hq, D), torch.bfloat16, "o")
    _chk(lse, (Hq, T), torch.float32, "lse")
    sc_ptr, sc_bytes = None, 0
    if for_backward:
        sc = plan.bwd_scratch()
        sc_ptr, sc_bytes = sc.data_ptr(), sc.numel()
    with torch.cuda.device(q.device):
        _check(lib().pp_attn_fwd(plan.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                 float(softmax_scale), o.data_ptr(), lse.data_ptr(), sc_ptr, sc_bytes,
                                 _stream()), "pp_attn_fwd")
    return o, lse


def pp_attn_bwd(plan: Plan, q, k, v, o, lse, d_o, softmax_scale: float, d_q=None, d_k=None, d_v=None,
                deterministic: bool = False):
    """``deterministic``: pp_attn_bwd_deterministic (bit-reproducible dQ; key tiles take turns)."""
    p = plan.problem
    T, Hq, Hkv, D = p.total_tokens, p.num_q_heads, p.num_kv_heads, p.head_dim
    _chk(q, (T, Hq, D), torch.bfloat16, "q")
    _chk(k, (T, Hkv, D), torch.bfloat16, "k")
    _chk(v, (T, Hkv, D), torch.bfloat16, "v")
    _chk(o, (T, Hq, D), torch.bfloat16, "o")
    _chk(d_o, (T, Hq, D), torch.bfloat16, "d_o")
    _chk(lse, (Hq, T), torch.float32, "lse")
    d_q = torch.empty_like(q) if d_q is None else d_q
    d_k = torch.empty_like(k) if d_k is None else d_k
    d_v = torch.empty_like(v) if d_v is None else d_v
    scratch = plan.bwd_scratch()
    fn = lib().pp_attn_bwd_deterministic if deterministic else lib().pp_attn_bwd
    with torch.cuda.device(q.device):
        _check(fn(plan.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                  o.data_ptr(), lse.data_ptr(), d_o.data_ptr(), float(softmax_scale),
                  d_q.data_ptr(), d_k.data_ptr(), d_v.data_ptr(), scratch.data_ptr(),
                  scratch.numel(), _stream()), "pp_attn_bwd")
    return d_q, d_k, d_v


def pp_position_ids(plan: Plan, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Packed position ids [T] int32: positions restart after the prompt for every response."""
    if out is None:
        out = torch.empty(plan.total_tokens, dtype=torch.int32, device=plan.workspace.device)
    _chk(out, (plan.total_tokens,), torch.int32, "position_ids")
    with torch.cuda.device(out.device):
        _check(lib().pp_position_ids(plan.handle, out.data_ptr(), _stream()), "pp_position_ids")
    return out


def pp_rope_qk(plan: Plan, q: torch.Tensor, k: torch.Tensor, rope_base: float = 10000.0):
    """Rotary embedding with the packed positions, in place on q [T,Hq,D] and k [T,Hkv,D]."""
    p = plan.problem
    _chk(q, (p.total_tokens, p.num_q_heads, p.head_dim), torch.bfloat16, "q")
    _chk(k, (p.total_tokens, p.num_kv_heads, p.head_dim), torch.bfloat16, "k")
    with torch.cuda.device(q.device):
        _check(lib().pp_rope_qk(plan.handle, q.data_ptr(), k.data_ptr(), float(rope_base), _stream()),
               "pp_rope_qk")
    return q, k


def pp_preference_loss(plan: Plan, token_logp: torch.Tensor, ref_token_logp: Optional[torch.Tensor],
                       beta: float, want_grad: bool = True):
    """Returns (resp_logp [N], resp_reward [N], grp_loss [G], d_token_logp [T] or None)."""
    p = plan.problem
    T, N, G = p.total_tokens, p.num_responses, p.num_groups
    _chk(token_logp, (T,), torch.float32, "token_logp")
    if ref_token_logp is not None:
        _chk(ref_token_logp, (T,), torch.float32, "ref_token_logp")
    dev = token_logp.device
    resp_logp = torch.empty(N, dtype=torch.float32, device=dev)
    resp_reward = torch.empty(N, dtype=torch.float32, device=dev)
    grp_loss = torch.empty(G, dtype=torch.float32, device=dev)
    grad = torch.empty(T, dtype=torch.float32, device=dev) if want_grad else None
    with torch.cuda.device(dev):
        _check(lib().pp_preference_loss(plan.handle, token_logp.data_ptr(),
                                        ref_token_logp.data_ptr() if ref_token_logp is not None else None,
                                        float(beta), resp_logp.data_ptr(), resp_reward.data_ptr(),
                                        grp_loss.data_ptr(), grad.data_ptr() if want_grad else None,
                                        _stream()), "pp_preference_loss")
    return resp_logp, resp_reward, grp_loss, grad


def pp_attn_bwd_noalloc_max_bytes() -> int:
    n = ctypes.c_size_t(0)
    _check(lib().pp_attn_bwd_noalloc_max_bytes(ctypes.byref(n)), "pp_attn_bwd_noalloc_max_bytes")
    return n.value


def pp_attn_bwd_noalloc(plan: Plan, q, k, v, o, lse, d_o, softmax_scale: float, d_q, d_k, d_v):
    """Backward for callers that must not allocate: the scratch is an array inside the
    library (32 MiB per GPU), so the outputs have to be passed in and nothing is allocated
    here either.  Problems whose scratch exceeds pp_attn_bwd_noalloc_max_bytes() raise
    PPError(-7).  Calls on one stream may follow each other; overlapping calls race."""
    p = plan.problem
    T, Hq, Hkv, D = p.total_tokens, p.num_q_heads, p.num_kv_heads, p.head_dim
    for t, shape, name in ((q, (T, Hq, D), "q"), (k, (T, Hkv, D), "k"), (v, (T, Hkv, D), "v"),
                           (o, (T, Hq, D), "o"), (d_o, (T, Hq, D), "d_o"), (d_q, (T, Hq, D), "d_q"),
                           (d_k, (T, Hkv, D), "d_k"), (d_v, (T, Hkv, D), "d_v")):
        _chk(t, shape, torch.bfloat16, name)
    _chk(lse, (Hq, T), torch.float32, "lse")
    with torch.cuda.device(q.device):
        _check(lib().pp_attn_bwd_noalloc(plan.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                         o.data_ptr(), lse.data_ptr(), d_o.data_ptr(),
                                         float(softmax_scale), d_q.data_ptr(), d_k.data_ptr(),
                                         d_v.data_ptr(), _stream()), "pp_attn_bwd_noalloc")
    return d_q, d_k, d_v


def pp_step_host_arena_bytes(problem: _Problem) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().pp_step_host_arena_bytes(ctypes.byref(problem), ctypes.byref(n)),
           "pp_step_host_arena_bytes")
    return n.value


def pp_step_host_runs(problem: _Problem) -> Tuple[np.ndarray, np.ndarray]:
    """(group_begin, token_begin) of the runs pp_attn_step_host cuts the problem into."""
    n = ctypes.c_int32(0)
    gb, tb = np.zeros(9, dtype=np.int32), np.zeros(9, dtype=np.int32)
    _check(lib().pp_step_host_runs(ctypes.byref(problem), ctypes.byref(n), gb.ctypes.data,
                                   tb.ctypes.data), "pp_step_host_runs")
    return gb[:n.value + 1], tb[:n.value + 1]


class HostStep:
    """pp_attn_step_host on page-locked host tensors: one whole pass (H2D copies, plan,
    forward, backward, D2H copies) enqueued on the current stream."""

    def __init__(self, workload, device: str = "cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("pp_attn_step_host needs a CUDA device (there is no CPU fallback)")
        w = workload
        self.scale = w.softmax_scale
        self.problem, self._keep = make_problem(w.descriptors(), w.num_q_heads, w.num_kv_heads,
                                                w.head_dim, w.total_tokens)
        self.arena = torch.empty(pp_step_host_arena_bytes(self.problem), dtype=torch.uint8,
                                 device=device)
        T, Hq, Hkv, D = w.total_tokens, w.num_q_heads, w.num_kv_heads, w.head_dim
        pin = lambda *shape, dtype=torch.bfloat16: torch.empty(*shape, dtype=dtype).pin_memory()
        self.o, self.dq = pin(T, Hq, D), pin(T, Hq, D)
        self.dk, self.dv = pin(T, Hkv, D), pin(T, Hkv, D)
        self.lse = pin(Hq, T, dtype=torch.float32)
        self.h2d_bytes = 2 * D * T * (2 * Hq + 2 * Hkv)
        self.d2h_bytes = 2 * D * T * (2 * Hq + 2 * Hkv) + 4 * Hq * T

    def __call__(self, q, k, v, d_o):
        """q, k, v, d_o: page-locked CPU bf16 tensors.  Results land in self.o, .lse, .dq, .dk,
        .dv once the current stream has been synchronised."""
        for t in (q, k, v, d_o):
            if t.is_cuda or not t.is_contiguous() or t.dtype != torch.bfloat16:
                raise ValueError("pp_attn_step_host takes contiguous CPU bf16 tensors")
        with torch.cuda.device(self.arena.device):
            _check(lib().pp_attn_step_host(ctypes.byref(self.problem), q.data_ptr(), k.data_ptr(),
                                           v.data_ptr(), d_o.data_ptr(), float(self.scale),
                                           self.o.data_ptr(), self.lse.data_ptr(), self.dq.data_ptr(),
                                           self.dk.data_ptr(), self.dv.data_ptr(),
                                           self.arena.data_ptr(), self.arena.numel(), _stream()),
                   "pp_attn_step_host")
        return self.o, self.lse, self.dq, self.dk, self.dv


def pp_profile_enable(on, backward_only: bool = False):
    """Kernel event timing: both main kernels, or only the backward main kernel."""
    global _profile_fwd
    mode = 0 if not on else (2 if backward_only else 1)
    _check(lib().pp_profile_enable(mode), "pp_profile_enable")
    _profile_fwd = mode == 1


_profile_fwd = False


def pp_profile_read() -> Tuple[Optional[float], float]:
    """(forward kernel ms or None, backward main kernel ms) of the latest calls; sync the stream first."""
    a, b = ctypes.c_float(0), ctypes.c_float(0)
    _check(lib().pp_profile_read(ctypes.byref(a) if _profile_fwd else None, ctypes.byref(b)),
           "pp_profile_read")
    return (a.value if _profile_fwd else None), b.value


def pp_profile_read_all(capacity: int = 64) -> Tuple[list, list]:
    """(forward kernel ms, backward main kernel ms) of the most recent calls since the last
    pp_profile_enable, oldest first (at most 64 each); sync the stream first."""
    a = (ctypes.c_float * capacity)()
    b = (ctypes.c_float * capacity)()
    na, nb = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(lib().pp_profile_read_all(a if _profile_fwd else None, b, capacity,
                                     ctypes.byref(na), ctypes.byref(nb)), "pp_profile_read_all")
    return ([a[i] for i in range(na.value)] if _profile_fwd else []), [b[i] for i in range(nb.value)]


def pp_last_launch_count() -> int:
    return int(lib().pp_last_launch_count())


def plan_for(workload, device: str = "cuda:0", desc_on_device: bool = False) -> Plan:
    """Convenience: plan of a :class:`workloads.Workload`."""
    return pp_build_plan(workload.descriptors(), workload.num_q_heads, workload.num_kv_heads,
                         workload.head_dim, workload.total_tokens, device, desc_on_device)


def pp_build_rows(grp_prompt_len: torch.Tensor, grp_resp_off: torch.Tensor, resp_len: torch.Tensor,
                  row_capacity: int):
    """Row builder (batch sorting + packing into rows of at most ``row_capacity`` tokens) on
    int32 DEVICE tensors.  Returns a dict of device tensors: order, row_group_off (trimmed to
    rows + 1), row_tokens, row_cost (trimmed to rows), grp_prompt_len, grp_resp_off, resp_len in
    row order, and ``status`` (code, detail) as Python ints (reading it synchronises)."""
    dev = grp_prompt_len.device
    G, N = int(grp_prompt_len.numel()), int(resp_len.numel())
    for t, n, name in ((grp_prompt_len, G, "grp_prompt_len"), (grp_resp_off, G + 1, "grp_resp_off"),
                       (resp_len, N, "resp_len")):
        _chk(t, (n,), torch.int32, name)
    nbytes = ctypes.c_size_t(0)
    _check(lib().pp_build_rows_workspace_bytes(G, ctypes.byref(nbytes)), "pp_build_rows_workspace_bytes")
    ws = torch.empty(nbytes.value, dtype=torch.uint8, device=dev)
    i32 = lambda n: torch.empty(n, dtype=torch.int32, device=dev)
    i64 = lambda n: torch.empty(n, dtype=torch.int64, device=dev)
    order, rgo, nrows, status = i32(G), i32(G + 1), i32(1), i32(2)
    rtok, rcost = i64(G), i64(G)
    oP, ooff, orl = i32(G), i32(G + 1), i32(N)
    with torch.cuda.device(dev):
        _check(lib().pp_build_rows(G, N, grp_prompt_len.data_ptr(), grp_resp_off.data_ptr(),
                                   resp_len.data_ptr(), int(row_capacity), ws.data_ptr(), ws.numel(),
                                   order.data_ptr(), rgo.data_ptr(), nrows.data_ptr(), rtok.data_ptr(),
                                   rcost.data_ptr(), oP.data_ptr(), ooff.data_ptr(), orl.data_ptr(),
                                   status.data_ptr(), _stream()), "pp_build_rows")
    st = status.tolist()
    r = int(nrows.item())
    return {"order": order, "row_group_off": rgo[:r + 1], "row_tokens": rtok[:r], "row_cost": rcost[:r],
            "grp_prompt_len": oP, "grp_resp_off": ooff, "resp_len": orl, "status": (st[0], st[1])}


def pp_assign_rows(row_cost: torch.Tensor, num_ranks: int):
    """Rows -> data-parallel ranks by longest-processing-time assignment on the attention cost.
    ``row_cost``: int64 DEVICE tensor [rows].  Returns device tensors (order [rows] int32,
    rank_of_row [rows] int32, rank_cost [num_ranks] int64)."""
    _chk(row_cost, (row_cost.numel(),), torch.int64, "row_cost")
    dev, R = row_cost.device, int(row_cost.numel())
    order = torch.empty(R, dtype=torch.int32, device=dev)
    rank_of_row = torch.empty(R, dtype=torch.int32, device=dev)
    rank_cost = torch.empty(int(num_ranks), dtype=torch.int64, device=dev)
    with torch.cuda.device(dev):
        _check(lib().pp_assign_rows(R, row_cost.data_ptr(), int(num_ranks), order.data_ptr(),
                                    rank_of_row.data_ptr(), rank_cost.data_ptr(), _stream()),
               "pp_assign_rows")
    return order, rank_of_row, rank_cost


def pp_debug_expire_wait(plan: Plan, site: int):
    """Test hook: lets one bounded wait run out on the plan's status word (see pp_attn.h)."""
    with torch.cuda.device(plan.workspace.device):
        _check(lib().pp_debug_expire_wait(plan.handle, int(site), _stream()), "pp_debug_expire_wait")
