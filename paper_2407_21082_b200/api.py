"""Python binding of the C ABI in include/eexit.h: argument marshalling only.

Tensors are torch CUDA tensors (torch supplies device memory and the current stream); bf16 tensors may be
passed as torch.bfloat16 or as int16/uint16 bit patterns.  Every function launches on torch's current
stream and returns without synchronising, exactly like the C calls underneath.
"""
from __future__ import annotations

import torch

from . import _lib

EE_PATH_AUTO, EE_PATH_STREAM, EE_PATH_TCGEN05, EE_PATH_SKINNY = 0, 1, 2, 3


class EExitError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = int(code)
        msg = _lib.load().ee_status_string(int(code)).decode()
        super().__init__(f"{where}: {msg} (ee_status {int(code)})")


def _check(code: int, where: str) -> None:
    if code != 0:
        raise EExitError(code, where)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _bf16(t: torch.Tensor) -> torch.Tensor:
    if t.dtype in (torch.int16, torch.uint16):
        t = t.view(torch.bfloat16)
    if t.dtype != torch.bfloat16:
        raise TypeError(f"expected bf16 (or its 16-bit patterns), got {t.dtype}")
    return t


def _dev(t: torch.Tensor, name: str) -> torch.Tensor:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    return t


def ee_exit_head_workspace_bytes(M: int, d: int, V: int) -> int:
    return int(_lib.load().ee_exit_head_workspace_bytes(int(M), int(d), int(V)))


def ee_exit_head_launches(M: int, d: int, V: int, path: int = EE_PATH_AUTO) -> int:
    return int(_lib.load().ee_exit_head_launches(int(M), int(d), int(V), int(path)))


def ee_workspace_init(workspace: torch.Tensor) -> None:
    _check(_lib.load().ee_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
           "ee_workspace_init")


def new_workspace(M: int, d: int, V: int, device="cuda") -> torch.Tensor:
    """Allocates (through torch) and initialises a workspace for ee_exit_head at these sizes."""
    nbytes = ee_exit_head_workspace_bytes(M, d, V)
    if nbytes == 0:
        raise EExitError(2, "ee_exit_head_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    ee_workspace_init(ws)
    return ws


def new_outputs(M: int, device="cuda") -> dict:
    return dict(argmax=torch.empty(M, dtype=torch.int32, device=device),
                entropy=torch.empty(M, dtype=torch.float32, device=device),
                maxprob=torch.empty(M, dtype=torch.float32, device=device),
                exit_mask=torch.empty(M, dtype=torch.uint8, device=device))


_OUT_DTYPES = dict(argmax=torch.int32, entropy=torch.float32, maxprob=torch.float32, exit_mask=torch.uint8)


def _check_head_tensors(h, gamma, beta, W, tau, out=None):
    """Host-side checks shared by the single-head wrappers: everything the kernels take on trust (shapes, strides,
    dtypes, devices) is verified here, so that a bad argument raises ValueError instead of reaching the device.
    Returns h and W as bf16 tensors and (M, d, V)."""
    h, W = _bf16(_dev(h, "h")), _bf16(_dev(W, "W"))
    if h.dim() != 2 or W.dim() != 2:
        raise ValueError("h must be [M, d] and W [V, d]")
    M, d = h.shape
    V = W.shape[0]
    if W.shape[1] != d or not W.is_contiguous() or (M > 0 and h.stride(1) != 1):
        raise ValueError("W must be contiguous [V, d] and h row-major [M, d]")
    for name, t in (("gamma", gamma), ("beta", beta)):
        if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and t.numel() == d):
            raise ValueError(f"{name} must be a contiguous float32 CUDA tensor of d = {d} elements")
        if t.device != h.device:
            raise ValueError(f"{name} is on {t.device}, h on {h.device}")
    if W.device != h.device:
        raise ValueError(f"W is on {W.device}, h on {h.device}")
    if isinstance(tau, torch.Tensor):
        if not (tau.is_cuda and tau.device == h.device and tau.dtype == torch.float32 and tau.is_contiguous() and tau.numel() == M):
            raise ValueError(f"a per-row tau must be a contiguous float32 CUDA tensor of M = {M} elements")
    if out is not None:
        for name, dtype in _OUT_DTYPES.items():
            t = out.get(name)
            if not (isinstance(t, torch.Tensor) and t.is_cuda and t.device == h.device and t.dtype == dtype and
                    t.is_contiguous() and t.numel() >= M):
                raise ValueError(f"out[{name!r}] must be a contiguous {dtype} CUDA tensor of at least M = {M} elements")
    return h, W, (M, d, V)


def _exit_head_args(h, gamma, beta, ln_eps, W, tau, out, workspace, path):
    h, W, (M, d, V) = _check_head_tensors(h, gamma, beta, W, tau, out)
    out = out if out is not None else new_outputs(M, h.device)
    workspace = workspace if workspace is not None else new_workspace(M, d, V, h.device)
    tau_t, tau_f = (tau, 0.0) if isinstance(tau, torch.Tensor) else (None, float(tau))
    args = (_ptr(h), h.stride(0) if M > 1 else max(h.stride(0), d), _ptr(gamma), _ptr(beta), float(ln_eps), _ptr(W),
            M, d, V, _ptr(tau_t), tau_f, _ptr(out["argmax"]), _ptr(out["entropy"]), _ptr(out["maxprob"]),
            _ptr(out["exit_mask"]), _ptr(workspace), workspace.numel(), _stream(), int(path))
    return args, out, (h, gamma, beta, W, tau_t, out, workspace)


def ee_exit_head(h, gamma, beta, ln_eps, W, tau, *, out=None, workspace=None, path=EE_PATH_AUTO) -> dict:
    """LayerNorm + exit-head projection + entropy / argmax / max-prob + exit decision for the rows of h.

    tau is a float (nats) or a float32 CUDA tensor [M] of per-row thresholds.  `out` (see new_outputs) and
    `workspace` (see new_workspace) are allocated when not given.
    """
    args, out, _ = _exit_head_args(h, gamma, beta, ln_eps, W, tau, out, workspace, path)
    _check(_lib.load().ee_exit_head_path(*args), "ee_exit_head")
    return out


class PreparedCall:
    """A C-ABI call with its arguments marshalled once, for loops that repeat the same call.

    Holds references to the tensors so that their memory stays alive; the stream is the one that was current
    at preparation time.  Calling it launches and returns, like the function it wraps.
    """
    __slots__ = ("_fn", "_args", "_where", "_keep", "out")

    def __init__(self, fn, args, where, keep, out):
        import ctypes as C
        self._fn = fn
        self._args = tuple(C.c_void_p(a) if (t is C.c_void_p) else t(a) for a, t in zip(args, fn.argtypes))
        self._where, self._keep, self.out = where, keep, out

    def __call__(self):
        code = self._fn(*self._args)
        if code:
            raise EExitError(code, self._where)
        return self.out


def ee_exit_head_multi_workspace_bytes(n_heads: int, M: int, d: int, V: int) -> int:
    return int(_lib.load().ee_exit_head_multi_workspace_bytes(int(n_heads), int(M), int(d), int(V)))


def ee_exit_head_multi_launches(n_heads: int, M: int, d: int, V: int) -> int:
    return int(_lib.load().ee_exit_head_multi_launches(int(n_heads), int(M), int(d), int(V)))


def _multi_args(heads, ln_eps, workspace):
    """heads: list of dicts with h, gamma, beta, W, tau and optionally out (see new_outputs)."""
    n = len(heads)
    arr = (_lib.EEHead * n)()
    keep, outs = [], []
    M, d = _bf16(heads[0]["h"]).shape
    V = heads[0]["W"].shape[0]
    for i, hd in enumerate(heads):
        h, W = _bf16(_dev(hd["h"], "h")), _bf16(_dev(hd["W"], "W"))
        if h.shape != (M, d) or W.shape != (V, d) or not W.is_contiguous() or h.stride(1) != 1:
            raise ValueError("all heads must share M, d, V; W contiguous [V, d]; h row-major [M, d]")
        out = hd.get("out") or new_outputs(M, h.device)
        tau = hd["tau"]
        tau_t, tau_f = (tau, 0.0) if isinstance(tau, torch.Tensor) else (None, float(tau))
        e = arr[i]
        e.h, e.ld_h, e.gamma, e.beta, e.W = _ptr(h), (h.stride(0) if M > 1 else max(h.stride(0), d)), _ptr(hd["gamma"]), _ptr(hd["beta"]), _ptr(W)
        e.tau_per_row, e.tau = _ptr(tau_t), tau_f
        e.argmax, e.entropy, e.maxprob, e.exit_mask = (_ptr(out[k]) for k in ("argmax", "entropy", "maxprob", "exit_mask"))
        keep.append((h, W, hd["gamma"], hd["beta"], tau_t, out))
        outs.append(out)
    if workspace is None:
        nbytes = ee_exit_head_multi_workspace_bytes(n, M, d, V)
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=heads[0]["h"].device)
        ee_workspace_init(workspace)
    args = (arr, n, float(ln_eps), M, d, V, _ptr(workspace), workspace.numel(), _stream())
    return args, outs, (arr, keep, workspace)


def ee_exit_head_multi(heads, ln_eps, *, workspace=None) -> list:
    """ee_exit_head for several heads on batches of the same shape in one call; returns one output dict per head."""
    args, outs, _ = _multi_args(heads, ln_eps, workspace)
    _check(_lib.load().ee_exit_head_multi(*args), "ee_exit_head_multi")
    return outs


class PreparedMulti:
    """ee_exit_head_multi for a loop that repeats the call: the host work (argument checks, tensor maps, launch shapes)
    is done once here (ee_exit_head_plan_init) and a call only launches (ee_exit_head_plan_run) on the stream that was
    current at preparation time.  More heads than a plan takes fall back to ee_exit_head_multi with its argument
    block built once."""
    __slots__ = ("_args", "_keep", "out", "_plan", "_stream", "_run")

    def __init__(self, heads, ln_eps, workspace=None):
        import ctypes as C
        self._args, self.out, self._keep = _multi_args(heads, ln_eps, workspace)
        self._plan = None
        arr, n, eps, M, d, V, ws, ws_bytes, stream = self._args
        if 1 <= n <= _lib.EE_PLAN_MAX_HEADS and M >= 1:
            self._plan = _lib.EEExitHeadPlan()
            _check(_lib.load().ee_exit_head_plan_init(C.byref(self._plan), arr, n, eps, M, d, V, ws, ws_bytes), "ee_exit_head_plan_init")
            self._stream = C.c_void_p(stream)
            self._plan = C.byref(self._plan), self._plan          # the reference passed to C, and the object it refers to
            self._run = _lib.load().ee_exit_head_plan_run

    def __call__(self):
        code = self._run(self._plan[0], self._stream) if self._plan is not None else _lib.load().ee_exit_head_multi(*self._args)
        if code:
            raise EExitError(code, "ee_exit_head_multi")
        return self.out


def ee_exit_head_top2(h, gamma, beta, ln_eps, W, tau, *, out=None, workspace=None) -> dict:
    """ee_exit_head plus out["top2gap"]: the difference between the two largest probabilities of every row."""
    h, W, (M, d, V) = _check_head_tensors(h, gamma, beta, W, tau, out)
    if out is None:
        out = new_outputs(M, h.device)
        out["top2gap"] = torch.empty(M, dtype=torch.float32, device=h.device)
    if workspace is None:
        workspace = new_workspace(M, d, V, h.device)
    tau_t, tau_f = (tau, 0.0) if isinstance(tau, torch.Tensor) else (None, float(tau))
    _check(_lib.load().ee_exit_head_top2(
        _ptr(h), h.stride(0) if M > 1 else max(h.stride(0), d), _ptr(gamma), _ptr(beta), float(ln_eps), _ptr(W), M, d, V,
        _ptr(tau_t), tau_f, _ptr(out["argmax"]), _ptr(out["entropy"]), _ptr(out["maxprob"]), _ptr(out["top2gap"]),
        _ptr(out["exit_mask"]), _ptr(workspace), workspace.numel(), _stream()), "ee_exit_head_top2")
    return out


def ee_exit_head_results_bytes(n_heads: int, M: int) -> int:
    return int(_lib.load().ee_exit_head_results_bytes(n_heads, M))


def results_views(block: torch.Tensor, n_heads: int, M: int) -> list:
    """Views (no copies) of a packed result block (uint8, host or device) as one output dict per head."""
    stride = ee_exit_head_results_bytes(1, M)
    outs = []
    for k in range(n_heads):
        b = block[k * stride:(k + 1) * stride]
        outs.append(dict(argmax=b[0:4 * M].view(torch.int32), entropy=b[4 * M:8 * M].view(torch.float32),
                         maxprob=b[8 * M:12 * M].view(torch.float32), exit_mask=b[12 * M:13 * M]))
    return outs


class PreparedMultiHost:
    """ee_exit_head_multi_host with its argument block built once.

    heads: list of dicts with gamma, beta, W, tau (device tensors / floats).  h_host: pinned bf16
    [n_heads, M, d].  The staging buffers and the pinned result block are created here, once; `out_host`
    and `out_dev` are per-head views into the packed result blocks.
    """
    __slots__ = ("_args", "_keep", "out_host", "out_dev", "h_dev", "h2d_bytes", "d2h_bytes", "_plan")

    def __init__(self, heads, ln_eps, h_host, workspace):
        n, (_, M, d) = len(heads), h_host.shape
        V = heads[0]["W"].shape[0]
        dev = workspace.device
        arr = (_lib.EEHead * n)()
        keep = []
        for i, hd in enumerate(heads):
            W = _bf16(_dev(hd["W"], "W"))
            tau = hd["tau"]
            tau_t, tau_f = (tau, 0.0) if isinstance(tau, torch.Tensor) else (None, float(tau))
            e = arr[i]
            e.gamma, e.beta, e.W, e.tau_per_row, e.tau = _ptr(hd["gamma"]), _ptr(hd["beta"]), _ptr(W), _ptr(tau_t), tau_f
            keep.append((W, hd["gamma"], hd["beta"], tau_t))
        import ctypes as C
        nbytes = ee_exit_head_results_bytes(n, M)
        self.h_dev = torch.empty((n, M, d), dtype=torch.bfloat16, device=dev)
        res_dev = torch.zeros(nbytes, dtype=torch.uint8, device=dev)
        res_host = torch.zeros(nbytes, dtype=torch.uint8).pin_memory()
        self.out_dev, self.out_host = results_views(res_dev, n, M), results_views(res_host, n, M)
        self.h2d_bytes, self.d2h_bytes = h_host.numel() * 2, nbytes
        self._args = (arr, n, float(ln_eps), M, d, V, _ptr(h_host), _ptr(self.h_dev), _ptr(res_host), _ptr(res_dev),
                      _ptr(workspace), workspace.numel(), _stream())
        self._keep = (arr, keep, h_host, res_dev, res_host, workspace)
        self._plan = None
        if 1 <= n <= _lib.EE_PLAN_MAX_HEADS and M >= 1:
            # the plan's heads read their rows from the staging buffer and write into the packed device results
            for i in range(n):
                e, o = arr[i], self.out_dev[i]
                e.h, e.ld_h = self.h_dev[i].data_ptr(), d
                e.argmax, e.entropy, e.maxprob, e.exit_mask = (_ptr(o[k]) for k in ("argmax", "entropy", "maxprob", "exit_mask"))
            plan = _lib.EEExitHeadPlan()
            _check(_lib.load().ee_exit_head_plan_init(C.byref(plan), arr, n, float(ln_eps), M, d, V, _ptr(workspace), workspace.numel()),
                   "ee_exit_head_plan_init")
            self._plan = (C.byref(plan), plan, C.c_void_p(_ptr(h_host)), C.c_void_p(_ptr(self.h_dev)), C.c_size_t(self.h2d_bytes),
                          C.c_void_p(_ptr(res_host)), C.c_void_p(_ptr(res_dev)), C.c_size_t(nbytes), C.c_void_p(_stream()))

    def __call__(self):
        if self._plan is not None:
            p = self._plan
            code = _lib.load().ee_exit_head_plan_run_host(p[0], p[2], p[3], p[4], p[5], p[6], p[7], p[8])
        else:
            code = _lib.load().ee_exit_head_multi_host(*self._args)
        if code:
            raise EExitError(code, "ee_exit_head_multi_host")
        return self.out_host


def prepare_exit_head(h, gamma, beta, ln_eps, W, tau, *, out=None, workspace=None, path=EE_PATH_AUTO) -> PreparedCall:
    """ee_exit_head with the arguments marshalled once; see PreparedCall."""
    args, out, keep = _exit_head_args(h, gamma, beta, ln_eps, W, tau, out, workspace, path)
    return PreparedCall(_lib.load().ee_exit_head_path, args, "ee_exit_head", keep, out)


EE_STATIC_MAX_ROWS = 32


def ee_exit_head_static(h, gamma, beta, ln_eps, W, tau, *, out: dict) -> dict:
    """ee_exit_head for callers that may not allocate: no workspace argument, at most EE_STATIC_MAX_ROWS rows.

    The library's built-in scratch array is used, so nothing is allocated by the call.  `out` must be given
    (see new_outputs) -- this wrapper creates no tensors either.  Calls sharing a GPU must not overlap.
    """
    h, W, (M, d, V) = _check_head_tensors(h, gamma, beta, W, tau, out)
    tau_t, tau_f = (tau, 0.0) if isinstance(tau, torch.Tensor) else (None, float(tau))
    _check(_lib.load().ee_exit_head_static(
        _ptr(h), h.stride(0) if M > 1 else max(h.stride(0), d), _ptr(gamma), _ptr(beta), float(ln_eps), _ptr(W),
        M, d, V, _ptr(tau_t), tau_f, _ptr(out["argmax"]), _ptr(out["entropy"]), _ptr(out["maxprob"]),
        _ptr(out["exit_mask"]), _stream()), "ee_exit_head_static")
    return out


def ee_exit_head_static_query_error() -> int:
    """ee_query_async_error for the built-in array of ee_exit_head_static: synchronises the current stream; 0, or
    EE_ERR_TIMEOUT after putting the array's control block back to its initial state."""
    return int(_lib.load().ee_exit_head_static_query_error(_stream()))


def ee_exit_head_static_selftest_timeout() -> None:
    """Makes one bounded wait give up against the built-in array (see include/eexit.h)."""
    _check(_lib.load().ee_exit_head_static_selftest_timeout(_stream()), "ee_exit_head_static_selftest_timeout")


def _exit_head_host_args(h_host, h_dev, gamma, beta, ln_eps, W, tau, out_host, out_dev, workspace):
    W = _bf16(W)
    M, d = h_host.shape
    tau_t, tau_f = (tau, 0.0) if isinstance(tau, torch.Tensor) else (None, float(tau))
    args = (_ptr(h_host), _ptr(h_dev), _ptr(gamma), _ptr(beta), float(ln_eps), _ptr(W), M, d, W.shape[0], _ptr(tau_t), tau_f,
            _ptr(out_host["argmax"]), _ptr(out_host["entropy"]), _ptr(out_host["maxprob"]), _ptr(out_host["exit_mask"]),
            _ptr(out_dev["argmax"]), _ptr(out_dev["entropy"]), _ptr(out_dev["maxprob"]), _ptr(out_dev["exit_mask"]),
            _ptr(workspace), workspace.numel(), _stream())
    return args, (h_host, h_dev, gamma, beta, W, tau_t, out_host, out_dev, workspace)


def ee_exit_head_host(h_host, h_dev, gamma, beta, ln_eps, W, tau, out_host: dict, out_dev: dict, workspace) -> None:
    """Host-buffer variant: copies h_host (pinned CPU tensor) in, runs the head, copies the outputs to out_host."""
    args, _ = _exit_head_host_args(h_host, h_dev, gamma, beta, ln_eps, W, tau, out_host, out_dev, workspace)
    _check(_lib.load().ee_exit_head_host(*args), "ee_exit_head_host")


def prepare_exit_head_host(h_host, h_dev, gamma, beta, ln_eps, W, tau, out_host, out_dev, workspace) -> PreparedCall:
    args, keep = _exit_head_host_args(h_host, h_dev, gamma, beta, ln_eps, W, tau, out_host, out_dev, workspace)
    return PreparedCall(_lib.load().ee_exit_head_host, args, "ee_exit_head_host", keep, out_host)


def ee_compact(exit_mask, h=None, *, gather=True, out=None) -> dict:
    """Indices (ascending) and count of the rows with exit_mask == 0, and a dense copy of their rows of h."""
    args, out, _ = _compact_args(exit_mask, h, gather, out)
    _check(_lib.load().ee_compact(*args), "ee_compact")
    return out


def prepare_compact(exit_mask, h=None, *, gather=True, out=None) -> PreparedCall:
    args, out, keep = _compact_args(exit_mask, h, gather, out)
    return PreparedCall(_lib.load().ee_compact, args, "ee_compact", keep, out)


def _compact_args(exit_mask, h, gather, out):
    M = exit_mask.numel()
    dev = exit_mask.device
    gather = gather and h is not None
    if gather:
        h = _bf16(_dev(h, "h"))
    d = h.shape[1] if h is not None else 0
    if out is None:
        out = dict(kept_idx=torch.empty(M, dtype=torch.int32, device=dev),
                   kept_count=torch.empty(1, dtype=torch.int32, device=dev))
        if gather:
            out["h_out"] = torch.empty((M, d), dtype=torch.bfloat16, device=dev)
    ld = (h.stride(0) if M > 1 else max(h.stride(0), d)) if gather else 0
    args = (_ptr(exit_mask), _ptr(h) if gather else None, ld, M, d, _ptr(out["kept_idx"]),
            _ptr(out["kept_count"]), _ptr(out.get("h_out")) if gather else None, _stream())
    return args, out, (exit_mask, h, out)


def dssd_accept(draft_tok, draft_exit_mask, verify_tok, *, out=None) -> dict:
    """Draft length, accepted prefix length and next token per sequence (see include/eexit.h)."""
    args, out, _ = _accept_args(draft_tok, draft_exit_mask, verify_tok, out)
    _check(_lib.load().dssd_accept(*args), "dssd_accept")
    return out


def prepare_accept(draft_tok, draft_exit_mask, verify_tok, *, out=None) -> PreparedCall:
    args, out, keep = _accept_args(draft_tok, draft_exit_mask, verify_tok, out)
    return PreparedCall(_lib.load().dssd_accept, args, "dssd_accept", keep, out)


def _compact_accept_args(exit_mask, h, draft_tok, draft_exit_mask, verify_tok, gather, out):
    c_args, c_out, c_keep = _compact_args(exit_mask, h, gather, None if out is None else out["compact"])
    a_args, a_out, a_keep = _accept_args(draft_tok, draft_exit_mask, verify_tok, None if out is None else out["accept"])
    return c_args[:-1] + a_args, dict(compact=c_out, accept=a_out), (c_keep, a_keep)


def ee_compact_accept(exit_mask, h, draft_tok, draft_exit_mask, verify_tok, *, gather=True, out=None) -> dict:
    """`ee_compact` and `dssd_accept` in one launch; returns dict(compact=..., accept=...) of their results."""
    args, out, _ = _compact_accept_args(exit_mask, h, draft_tok, draft_exit_mask, verify_tok, gather, out)
    _check(_lib.load().ee_compact_accept(*args), "ee_compact_accept")
    return out


def prepare_compact_accept(exit_mask, h, draft_tok, draft_exit_mask, verify_tok, *, gather=True, out=None) -> PreparedCall:
    args, out, keep = _compact_accept_args(exit_mask, h, draft_tok, draft_exit_mask, verify_tok, gather, out)
    return PreparedCall(_lib.load().ee_compact_accept, args, "ee_compact_accept", keep, out)


def ee_cascade_workspace_bytes(M: int, d: int, V: int) -> int:
    return int(_lib.load().ee_cascade_workspace_bytes(int(M), int(d), int(V)))


def ee_calibrate_workspace_bytes(n: int) -> int:
    return int(_lib.load().ee_calibrate_workspace_bytes(int(n)))


def ee_head_kl_workspace_bytes(M: int, d: int, V: int) -> int:
    return int(_lib.load().ee_head_kl_workspace_bytes(int(M), int(d), int(V)))


def _head_kl_args(head, teacher, ln_eps, out, workspace, labels=None):
    hh, Wh = _bf16(_dev(head["h"], "h")), _bf16(_dev(head["W"], "W"))
    ht, Wt = _bf16(_dev(teacher["h"], "h")), _bf16(_dev(teacher["W"], "W"))
    M, d = hh.shape
    V = Wh.shape[0]
    if ht.shape != (M, d) or Wt.shape != (V, d) or not (Wh.is_contiguous() and Wt.is_contiguous()):
        raise ValueError("head and teacher must share M, d, V; W contiguous [V, d]")
    dev = hh.device
    if out is None:
        out = dict(kl=torch.empty(M, dtype=torch.float32, device=dev), loss=torch.zeros(2, dtype=torch.float32, device=dev))
        if labels is not None:
            out["ce"] = torch.empty(M, dtype=torch.float32, device=dev)
    if labels is not None and (labels.dtype != torch.int32 or not labels.is_contiguous() or labels.numel() != M):
        raise TypeError("labels must be a contiguous int32 tensor [M]")
    if workspace is None:
        workspace = torch.empty(int(_lib.load().ee_head_kl_workspace_bytes(M, d, V)), dtype=torch.uint8, device=dev)
        ee_workspace_init(workspace)

    def ld(h):
        return h.stride(0) if M > 1 else max(h.stride(0), d)

    args = (_ptr(hh), ld(hh), _ptr(head["gamma"]), _ptr(head["beta"]), _ptr(Wh), _ptr(ht), ld(ht), _ptr(teacher["gamma"]),
            _ptr(teacher["beta"]), _ptr(Wt), float(ln_eps), M, d, V, _ptr(labels), _ptr(out["kl"]),
            _ptr(out.get("ce")) if labels is not None else None, _ptr(out.get("loss")), _ptr(workspace), workspace.numel(), _stream())
    return args, out, (hh, Wh, ht, Wt, head, teacher, workspace, out, labels)


def ee_head_kl(head, teacher, ln_eps, *, labels=None, out=None, workspace=None) -> dict:
    """KL divergence of a head's distribution from the teacher's, per token and mean (see include/eexit.h); with
    `labels` also the cross-entropy per token (out["ce"]) and its mean (out["loss"][1]).
    head / teacher: dicts with h, gamma, beta, W."""
    args, out, _ = _head_kl_args(head, teacher, ln_eps, out, workspace, labels)
    _check(_lib.load().ee_head_kl(*args), "ee_head_kl")
    return out


def prepare_head_kl(head, teacher, ln_eps, *, labels=None, out=None, workspace=None) -> PreparedCall:
    args, out, keep = _head_kl_args(head, teacher, ln_eps, out, workspace, labels)
    return PreparedCall(_lib.load().ee_head_kl, args, "ee_head_kl", keep, out)


def ee_selftest_wait_timeout(workspace) -> None:
    """Makes one bounded device-side wait give up (see include/eexit.h); ee_query_async_error then reports it."""
    _check(_lib.load().ee_selftest_wait_timeout(_ptr(workspace), workspace.numel(), _stream()), "ee_selftest_wait_timeout")


def ee_selftest_read_stream(buffer, workspace) -> None:
    """Reads `buffer` (a device tensor) once with the kernels' weight-streaming mechanism (see include/eexit.h);
    the caller times it."""
    _check(_lib.load().ee_selftest_read_stream(_ptr(buffer), buffer.numel() * buffer.element_size(), _ptr(workspace),
                                               workspace.numel(), _stream()), "ee_selftest_read_stream")


def _cascade_args(heads, ln_eps, out, workspace):
    n = len(heads)
    arr = (_lib.EEHead * n)()
    keep = []
    M, d = _bf16(heads[0]["h"]).shape
    V = heads[0]["W"].shape[0]
    dev = heads[0]["h"].device
    for i, hd in enumerate(heads):
        h, W = _bf16(_dev(hd["h"], "h")), _bf16(_dev(hd["W"], "W"))
        if h.shape != (M, d) or W.shape != (V, d) or not W.is_contiguous() or h.stride(1) != 1:
            raise ValueError("all heads must share M, d, V; W contiguous [V, d]; h row-major [M, d]")
        e = arr[i]
        e.h, e.ld_h, e.gamma, e.beta, e.W = _ptr(h), (h.stride(0) if M > 1 else max(h.stride(0), d)), _ptr(hd["gamma"]), _ptr(hd["beta"]), _ptr(W)
        e.tau_per_row, e.tau = None, float(hd["tau"])
        keep.append((h, W, hd["gamma"], hd["beta"]))
    if out is None:
        out = dict(exit_head=torch.empty(M, dtype=torch.int32, device=dev), token=torch.empty(M, dtype=torch.int32, device=dev),
                   entropy=torch.empty(M, dtype=torch.float32, device=dev), rows_in=torch.empty(n, dtype=torch.int32, device=dev))
    if workspace is None:
        workspace = torch.empty(int(_lib.load().ee_cascade_workspace_bytes(M, d, V)), dtype=torch.uint8, device=dev)
        ee_workspace_init(workspace)
    args = (arr, n, float(ln_eps), M, d, V, _ptr(out["exit_head"]), _ptr(out["token"]), _ptr(out["entropy"]), _ptr(out["rows_in"]),
            _ptr(workspace), workspace.numel(), _stream())
    return args, out, (arr, keep, workspace, out)


def ee_cascade(heads, ln_eps, *, out=None, workspace=None) -> dict:
    """Cascade of heads on a batch (see include/eexit.h): heads is a list of dicts with h, gamma, beta, W, tau."""
    args, out, _ = _cascade_args(heads, ln_eps, out, workspace)
    _check(_lib.load().ee_cascade(*args), "ee_cascade")
    return out


class PreparedCascade:
    """ee_cascade with its argument block built once (see PreparedCall)."""
    __slots__ = ("_args", "_keep", "out")

    def __init__(self, heads, ln_eps, out=None, workspace=None):
        self._args, self.out, self._keep = _cascade_args(heads, ln_eps, out, workspace)

    def __call__(self):
        code = _lib.load().ee_cascade(*self._args)
        if code:
            raise EExitError(code, "ee_cascade")
        return self.out


def _calibrate_args(entropy, argmax_head, argmax_final, epsilon, out, workspace):
    n = entropy.numel()
    dev = entropy.device
    if not (entropy.dtype == torch.float32 and argmax_head.dtype == torch.int32 and argmax_final.dtype == torch.int32):
        raise TypeError("entropy must be float32, the argmax arrays int32")
    if not (entropy.is_contiguous() and argmax_head.is_contiguous() and argmax_final.is_contiguous()):
        raise ValueError("calibration arrays must be contiguous")
    if out is None:
        out = dict(tau=torch.empty(1, dtype=torch.float32, device=dev), counts=torch.empty(3, dtype=torch.int32, device=dev))
    if workspace is None:
        workspace = torch.empty(int(_lib.load().ee_calibrate_workspace_bytes(n)), dtype=torch.uint8, device=dev)
    args = (_ptr(entropy), _ptr(argmax_head), _ptr(argmax_final), n, float(epsilon), _ptr(out["tau"]), _ptr(out["counts"]),
            _ptr(workspace), workspace.numel(), _stream())
    return args, out, (entropy, argmax_head, argmax_final, workspace, out)


def ee_calibrate(entropy, argmax_head, argmax_final, epsilon, *, out=None, workspace=None) -> dict:
    """Threshold of one head from a calibration set (see include/eexit.h): dict(tau [1], counts [3]) on the device."""
    args, out, _ = _calibrate_args(entropy, argmax_head, argmax_final, epsilon, out, workspace)
    _check(_lib.load().ee_calibrate(*args), "ee_calibrate")
    return out


def prepare_calibrate(entropy, argmax_head, argmax_final, epsilon, *, out=None, workspace=None) -> PreparedCall:
    args, out, keep = _calibrate_args(entropy, argmax_head, argmax_final, epsilon, out, workspace)
    return PreparedCall(_lib.load().ee_calibrate, args, "ee_calibrate", keep, out)


def dssd_commit(draft_tok, draft_exit_mask, verify_tok, eos_token, state: dict, *, out=None) -> dict:
    """Commit step of a DSSD round (see include/eexit.h).  `state` holds the sequences' device tensors: out_tok
    int32 [S, capacity], seq_len int32 [S], finished uint8 [S], stats int64 [4]; they are updated in place."""
    S, k = draft_tok.shape
    kv = verify_tok.shape[1]
    dev = draft_tok.device
    if not (draft_tok.is_contiguous() and verify_tok.is_contiguous() and state["out_tok"].is_contiguous()):
        raise ValueError("token arrays must be contiguous")
    if out is None:
        out = {n: torch.empty(S, dtype=torch.int32, device=dev) for n in ("draft_len", "accept_len", "next_tok")}
    _check(_lib.load().dssd_commit(_ptr(draft_tok), _ptr(draft_exit_mask), _ptr(verify_tok), S, k, kv, int(eos_token),
                                   _ptr(state["out_tok"]), state["out_tok"].shape[1], _ptr(state["seq_len"]),
                                   _ptr(state["finished"]), _ptr(out["draft_len"]), _ptr(out["accept_len"]),
                                   _ptr(out["next_tok"]), _ptr(state["stats"]), _stream()), "dssd_commit")
    return out


class TableModel:
    """Stand-in model for dssd_round served by the library itself (ee_hidden_from_tables in include/eexit.h): the
    hidden state after a token is that token's row of a table, one table per draft head's layer (`draft_table`: a
    tensor, or a list of K tensors, shallowest first) and `verify_table` for the verification pass, bf16 [V, d]
    device tensors.  Pass it to DssdRound as `hidden_fn`.  chained=True launches its kernel with programmatic stream
    serialization (early trigger, wait before the tokens are read)."""

    def __init__(self, draft_table, verify_table, chained: bool = False):
        drafts = list(draft_table) if isinstance(draft_table, (list, tuple)) else [draft_table]
        self.tables = tuple(_bf16(_dev(t, "table")) for t in drafts + [verify_table])
        if len(drafts) > _lib.EE_ROUND_MAX_DRAFT_HEADS:
            raise ValueError(f"at most {_lib.EE_ROUND_MAX_DRAFT_HEADS} draft tables")
        if any(t.shape != self.tables[0].shape for t in self.tables) or not all(t.is_contiguous() for t in self.tables):
            raise ValueError("tables must be contiguous and of one shape [V, d]")
        V, d = self.tables[0].shape
        self.struct = _lib.EEHiddenTables()
        for i, t in enumerate(self.tables):
            self.struct.table[i] = _ptr(t)
        self.struct.d, self.struct.V, self.struct.chained = d, V, int(bool(chained))


class DssdRound:
    """dssd_round (see include/eexit.h) with its argument block built once.

    draft_head: a dict with gamma, beta, W, tau, or a list of K such dicts (shallowest head first: per position the
    first confident one supplies the token); verify_head: dict with gamma, beta, W.  hidden_fn(tokens, which, h_out) is
    the caller's model: `tokens` int32 [n_rows] and `h_out` bf16 [n_rows, d] are device tensors (views into the
    workspace); it must fill h_out on the current stream with the hidden states at draft head `which`'s layer
    (which < K) or the full model's (which = K).  all_layers=True asks for ONE call per drafting step instead of K:
    which = -1 and h_out bf16 [K, n_rows, d], layer by layer (the library's TableModel is always driven that way).
    `state`: last_tok, out_tok, seq_len, finished, stats.  With a list
    of heads, self.head_use (int64 [K]) accumulates the positions each head supplied."""

    def __init__(self, draft_head, verify_head, ln_eps, k, eos_token, hidden_fn, state, workspace=None, all_layers=None):
        import ctypes as C
        S = state["last_tok"].numel()
        multi = isinstance(draft_head, (list, tuple))
        drafts = list(draft_head) if multi else [draft_head]
        K = len(drafts)
        Wd = [_bf16(_dev(h["W"], "W")) for h in drafts]
        Wv = _bf16(_dev(verify_head["W"], "W"))
        V, d = Wd[0].shape
        dev = Wd[0].device
        if workspace is None:
            workspace = torch.empty(int(_lib.load().dssd_round_multi_workspace_bytes(S, k, d, V, K)), dtype=torch.uint8, device=dev)
            ee_workspace_init(workspace)
        self.workspace, self.state = workspace, state
        self.out = {n: torch.empty(S, dtype=torch.int32, device=dev) for n in ("draft_len", "accept_len", "next_tok")}
        self.head_use = torch.zeros(K, dtype=torch.int64, device=dev) if multi else None
        base = workspace.data_ptr()

        def trampoline(user, tokens_ptr, n_rows, which, h_ptr, stream):
            try:
                tokens = workspace[tokens_ptr - base:tokens_ptr - base + 4 * n_rows].view(torch.int32)
                layers = K if which < 0 else 1
                h_out = workspace[h_ptr - base:h_ptr - base + 2 * layers * n_rows * d].view(torch.bfloat16)
                h_out = h_out.view(K, n_rows, d) if which < 0 else h_out.view(n_rows, d)
                hidden_fn(tokens, which, h_out)
                return 0
            except Exception:                    # an exception must not cross the C boundary
                import traceback
                traceback.print_exc()
                return 1

        native = isinstance(hidden_fn, TableModel)
        if native and (hidden_fn.tables[0].shape != (V, d) or len(hidden_fn.tables) != K + 1):
            raise ValueError("the table model needs one [V, d] table per draft head and one for the verification pass")
        self._cb = C.cast(_lib.load().ee_hidden_from_tables, _lib.HIDDEN_FN) if native else _lib.HIDDEN_FN(trampoline)
        a = _lib.EEDssdRoundArgs()
        a.S, a.k, a.d, a.V, a.ln_eps, a.eos_token = S, int(k), d, V, float(ln_eps), int(eos_token)
        arr = (_lib.EEHead * K)()
        for dst, src, W in [(arr[i], drafts[i], Wd[i]) for i in range(K)] + [(a.draft_head, drafts[0], Wd[0]), (a.verify_head, verify_head, Wv)]:
            dst.gamma, dst.beta, dst.W, dst.tau = _ptr(src["gamma"]), _ptr(src["beta"]), _ptr(W), float(src.get("tau", 0.0))
        if multi:
            a.n_draft_heads, a.draft_heads, a.head_use = K, arr, _ptr(self.head_use)
        a.hidden, a.hidden_user = self._cb, (C.cast(C.pointer(hidden_fn.struct), C.c_void_p) if native else None)
        a.hidden_all_layers = int(native if all_layers is None else bool(all_layers))
        a.last_tok, a.out_tok, a.capacity = _ptr(state["last_tok"]), _ptr(state["out_tok"]), state["out_tok"].shape[1]
        a.seq_len, a.finished, a.stats = _ptr(state["seq_len"]), _ptr(state["finished"]), _ptr(state["stats"])
        a.draft_len, a.accept_len, a.next_tok = (_ptr(self.out[n]) for n in ("draft_len", "accept_len", "next_tok"))
        a.workspace, a.workspace_bytes, a.stream = _ptr(workspace), workspace.numel(), _stream()
        self._args, self._keep = a, (Wd, Wv, drafts, verify_head, C, hidden_fn, arr)

    def __call__(self):
        import ctypes as C
        code = _lib.load().dssd_round(C.byref(self._args))
        if code:
            raise EExitError(code, "dssd_round")
        return self.out


def _accept_args(draft_tok, draft_exit_mask, verify_tok, out):
    S, k = draft_tok.shape
    kv = verify_tok.shape[1]
    dev = draft_tok.device
    if not (draft_tok.is_contiguous() and verify_tok.is_contiguous()):
        raise ValueError("token arrays must be contiguous")
    if out is None:
        out = {n: torch.empty(S, dtype=torch.int32, device=dev) for n in ("draft_len", "accept_len", "next_tok")}
    args = (_ptr(draft_tok), _ptr(draft_exit_mask), _ptr(verify_tok), S, k, kv,
            _ptr(out["draft_len"]), _ptr(out["accept_len"]), _ptr(out["next_tok"]), _stream())
    return args, out, (draft_tok, draft_exit_mask, verify_tok, out)


def ee_query_async_error(workspace) -> int:
    """Synchronises the current stream; 0 if no bounded wait gave up since the last query, else EE_ERR_TIMEOUT."""
    return int(_lib.load().ee_query_async_error(_ptr(workspace), _stream()))
