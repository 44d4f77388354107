"""ctypes binding of include/sparse_ffn.h.  Marshals torch tensors into plain pointers."""
from __future__ import annotations

import ctypes
import os
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
ACT = {"relu": 0, "sqrelu": 1, "rsplus": 2}
ACT_UP = dict(ACT, silu=4)  # activations of the up projection (double activation); SILU is not a gate activation
PATH = {"auto": 0, "general": 1, "fused": 2, "mma_sync": 3}
_STATUS = {0: "ok", 1: "invalid argument", 2: "unsupported shape, alignment or path",
           3: "workspace missing, misaligned or too small", 4: "CUDA runtime error",
           5: "device-side bounded wait ran out", 6: "debug build: index outside its array"}


class SFFNError(RuntimeError):
    def __init__(self, where: str, code: int):
        detail = ""
        if code == 4 and _lib is not None:
            detail = ": " + _lib.sffn_last_cuda_error().decode()
        super().__init__(f"{where}: status {code} ({_STATUS.get(code, 'unknown')}{detail})")
        self.code = code


class _Gate(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("r", ctypes.c_int32), ("W_g", ctypes.c_void_p),
                ("V", ctypes.c_void_p), ("U", ctypes.c_void_p), ("g_idx", ctypes.c_void_p),
                ("g_sign", ctypes.c_void_p), ("rms_gain", ctypes.c_void_p),
                ("use_rmsnorm", ctypes.c_int32), ("rms_eps", ctypes.c_float)]


class _Q8Scales(ctypes.Structure):
    _fields_ = [("s_gate", ctypes.c_void_p), ("s_V", ctypes.c_void_p), ("s_up", ctypes.c_void_p),
                ("s_down", ctypes.c_void_p)]


def lib_path() -> Path:
    """The library this process loads: libsparse_ffn.so, or the build named by SFFN_LIBRARY (e.g. the time-stamp
    build libsparse_ffn_trace.so)."""
    import os

    return _PKG / os.environ.get("SFFN_LIBRARY", "libsparse_ffn.so")


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is None:
        p = lib_path()
        if not p.exists():
            raise RuntimeError(f"{p} is missing: build it with `python -m paper_2609_31975_b200.build` "
                               "(the sparse FFN has no CPU or PyTorch fallback)")
        lib = ctypes.CDLL(str(p))
        vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        lib.sffn_workspace_bytes.argtypes = [i, i, i, i, i, ctypes.POINTER(sz)]
        lib.sffn_create.argtypes = [ctypes.POINTER(vp), i, i, i, i, i, vp, sz]
        lib.sffn_destroy.argtypes = [vp]
        lib.sffn_set_path.argtypes = [vp, i]
        lib.sffn_set_up_activation.argtypes = [vp, i]
        lib.sffn_set_gated_skip.argtypes = [vp, i]
        lib.sffn_set_gate_engine.argtypes = [vp, i]
        fwd = [vp, vp, i, ctypes.POINTER(_Gate), vp, vp, vp, i, vp, vp]
        lib.sparse_ffn_forward.argtypes = fwd
        lib.dense_ffn_forward.argtypes = fwd
        lib.sparse_ffn_forward_host.argtypes = fwd
        fwd_q8 = [vp, vp, i, ctypes.POINTER(_Gate), vp, vp, vp, ctypes.POINTER(_Q8Scales), i, vp, vp]
        lib.sparse_ffn_forward_q8.argtypes = fwd_q8
        lib.dense_ffn_forward_q8.argtypes = fwd_q8
        lib.sparse_ffn_forward_q4.argtypes = fwd_q8
        lib.dense_ffn_forward_q4.argtypes = fwd_q8
        lib.sffn_last_active.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), vp]
        lib.sffn_last_device_status.argtypes = [vp, ctypes.POINTER(i)]
        lib.sffn_launch_count.argtypes = [vp, ctypes.POINTER(ctypes.c_longlong)]
        lib.sparse_ffn_forward_static.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, vp, vp]
        lib.sffn_status_string.argtypes = [i]
        lib.sffn_residual_cast.argtypes = [vp, vp, ctypes.c_float, vp, i, i, vp]
        lib.sffn_status_string.restype = ctypes.c_char_p
        lib.sffn_lopa_m_step.argtypes = [vp, vp, i, i, vp, vp, vp, vp, vp]
        lib.sffn_lopa_residual.argtypes = [vp, vp, vp, i, i, vp, vp]
        lib.sffn_last_cuda_error.argtypes = []
        lib.sffn_last_cuda_error.restype = ctypes.c_char_p
        lib.sffn_test_set_knob.argtypes = [i, ctypes.c_longlong]
        lib.sffn_reset.argtypes = [vp, vp]
        _lib = lib
    return _lib


GATE_ENGINE = {"auto": 0, "cuda_core": 1, "tensor_core": 2}
KNOB = {"pdl": 0, "tensor_gate": 1, "wait_cycles": 2, "skip_arrival_cta": 3, "ring_gate_slots": 4,
        "ring_act_slots": 5, "trace_buffer": 6, "ring_parked_stages": 7, "l2_hints": 8, "drop_stage": 9,
        "poison_list": 10}


def test_set_knob(name: str, value: int):
    """Process-wide test hook of the library (see the "test hooks" section of sparse_ffn.h)."""
    _check("sffn_test_set_knob", load_library().sffn_test_set_knob(KNOB[name], int(value)))


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _codes(m):
    """The tensor whose address goes to the library: a quantised matrix given as dict(q=codes, s=row scales), or a tensor."""
    if isinstance(m, dict):
        q, s = m["q"], m["s"]
        if q.dtype not in (torch.int8, torch.uint8) or s.dtype != torch.float32 or s.shape != (q.shape[0],):
            raise TypeError("a quantised matrix is dict(q=int8 [rows, cols] or packed 4-bit uint8 [rows, cols / 2], "
                            "s=float32 [rows])")
        return q
    return m


def _check(where: str, rc: int):
    if rc != 0:
        raise SFFNError(where, rc)


def sparse_ffn_forward_static(x, W_g, b_g, W_up, W_down, act="relu", y=None, stream=None):
    """Handle-free, allocation-free variant (standard gate, one token): the library's built-in
    scratch array replaces the workspace.  For callers that cannot allocate device memory at call
    time; shapes are limited to D <= 8192, H <= 32768, and calls that may overlap on the GPU must be
    serialised by the caller (they share the scratch).  `y` must be supplied by such a caller; it
    is created here only as a convenience for tests."""
    lib = load_library()
    H, D = W_up.shape
    if y is None:
        y = torch.empty(D, dtype=torch.float32, device=x.device)
    s = torch.cuda.current_stream(x.device) if stream is None else stream
    _check("sparse_ffn_forward_static",
           lib.sparse_ffn_forward_static(_ptr(x), _ptr(W_g), _ptr(b_g), _ptr(W_up), _ptr(W_down), D, H,
                                         1 if W_up.dtype == torch.bfloat16 else 0,
                                         ACT[act] if isinstance(act, str) else int(act), _ptr(y),
                                         ctypes.c_void_p(s.cuda_stream)))
    return y


def residual_cast(y, resid, alpha, out, stream=None):
    """out = dtype(resid + alpha * y) for an fp32 FFN output ``y`` (glue between the FFN calls of a layer loop)."""
    lib = load_library()
    assert y.dtype == torch.float32 and resid.dtype == out.dtype and y.numel() == resid.numel() == out.numel()
    s = stream if stream is not None else torch.cuda.current_stream(y.device)
    _check("sffn_residual_cast",
           lib.sffn_residual_cast(_ptr(y), _ptr(resid), float(alpha), _ptr(out), y.numel(),
                                  1 if out.dtype == torch.bfloat16 else 0, ctypes.c_void_p(s.cuda_stream)))
    return out


def lopa_m_step(W, P=None, stream=None):
    """M-step of the LoPA approximation (Sec. 3.4) on fp32 device tensors: per row of R = W - P the column of the
    largest |R_ij| and its sign.  Returns (g_idx int32 [H], g_sign int8 [H], row_energy float64 [H], row_best fp32 [H])."""
    lib = load_library()
    if W.dtype != torch.float32 or not W.is_cuda or not W.is_contiguous() or W.dim() != 2:
        raise TypeError("W must be a contiguous fp32 CUDA matrix")
    if P is not None and (P.dtype != torch.float32 or P.shape != W.shape or not P.is_contiguous()):
        raise TypeError("P must match W")
    H, D = W.shape
    g_idx = torch.empty(H, dtype=torch.int32, device=W.device)
    g_sign = torch.empty(H, dtype=torch.int8, device=W.device)
    energy = torch.empty(H, dtype=torch.float64, device=W.device)
    best = torch.empty(H, dtype=torch.float32, device=W.device)
    s = torch.cuda.current_stream(W.device) if stream is None else stream
    _check("sffn_lopa_m_step", lib.sffn_lopa_m_step(_ptr(W), _ptr(P), H, D, _ptr(g_idx), _ptr(g_sign), _ptr(energy),
                                                    _ptr(best), ctypes.c_void_p(s.cuda_stream)))
    return g_idx, g_sign, energy, best


def lopa_residual(W, g_idx, g_sign, stream=None):
    """A = W - M for the one-nonzero-per-row matrix M described by (g_idx, g_sign); fp32 device tensors."""
    lib = load_library()
    H, D = W.shape
    A = torch.empty_like(W)
    s = torch.cuda.current_stream(W.device) if stream is None else stream
    _check("sffn_lopa_residual", lib.sffn_lopa_residual(_ptr(W), _ptr(g_idx), _ptr(g_sign), H, D, _ptr(A),
                                                        ctypes.c_void_p(s.cuda_stream)))
    return A


class SparseFFN:
    """One library handle (fixed D, H, dtype, limits r_max and B_max) plus its torch-owned workspace.

    ``gate`` arguments are dicts: ``{"W_g": t}`` for standard gating, or
    ``{"V": t, "U": t, "g_idx": t|None, "g_sign": t|None, "rms_gain": t|None,
    "use_rmsnorm": bool, "rms_eps": float}`` for the LoPA gate.

    Weight-only int8: hand every weight matrix (W_up, W_down and W_g, or V and U inside ``gate``) as
    ``dict(q=int8 codes [rows, cols], s=float32 row scales [rows])`` to the ``*_q8`` methods (or to
    :meth:`prepared`); the handle's dtype, the tokens', must then be bfloat16.
    """

    def __init__(self, D: int, H: int, dtype: torch.dtype, r_max: int = 0, B_max: int = 1,
                 device="cuda:0"):
        if dtype not in (torch.float32, torch.bfloat16):
            raise TypeError("dtype must be torch.float32 or torch.bfloat16")
        self.lib = load_library()
        self.D, self.H, self.dtype, self.r_max, self.B_max = D, H, dtype, r_max, B_max
        self.device = torch.device(device)
        self._dt = 1 if dtype == torch.bfloat16 else 0
        need = ctypes.c_size_t(0)
        _check("sffn_workspace_bytes", self.lib.sffn_workspace_bytes(D, H, r_max, B_max, self._dt, ctypes.byref(need)))
        self.workspace_bytes = need.value
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(need.value + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            h = ctypes.c_void_p()
            _check("sffn_create", self.lib.sffn_create(ctypes.byref(h), D, H, r_max, B_max, self._dt,
                                                       ctypes.c_void_p(self._ws_ptr), need.value))
        self._h = h
        if os.environ.get("SFFN_GATED_SKIP") == "1":   # lets a profiler run of bench.py take the gated variant
            self.set_gated_skip(True)
        self._keep = None

    def close(self):
        if getattr(self, "_h", None):
            self.lib.sffn_destroy(self._h)
            self._h = None

    __del__ = close

    def set_up_activation(self, act_up):
        """Double activation: ``act_up`` in ACT (or None for Eq. 1) is applied to the up projection."""
        code = 3 if act_up is None else ACT_UP[act_up]
        _check("sffn_set_up_activation", self.lib.sffn_set_up_activation(self._h, code))

    def set_gated_skip(self, on: bool):
        """Single-token double-activation calls fetch W_down rows only where h != 0 (sffn_set_gated_skip; default off)."""
        _check("sffn_set_gated_skip", self.lib.sffn_set_gated_skip(self._h, 1 if on else 0))

    def set_path(self, path: str):
        _check("sffn_set_path", self.lib.sffn_set_path(self._h, PATH[path]))

    def set_gate_engine(self, engine: str):
        """Where single-token calls compute the gate: "auto", "cuda_core" or "tensor_core" (sffn_set_gate_engine)."""
        _check("sffn_set_gate_engine", self.lib.sffn_set_gate_engine(self._h, GATE_ENGINE[engine]))

    def _gate(self, gate: dict) -> _Gate:
        g = _Gate()
        if "W_g" in gate:
            g.kind, g.W_g = 0, _codes(gate["W_g"]).data_ptr()
        else:
            g.kind, g.r = 1, _codes(gate["V"]).shape[0]
            g.V, g.U = _codes(gate["V"]).data_ptr(), _codes(gate["U"]).data_ptr()
            for k in ("g_idx", "g_sign", "rms_gain"):
                t = gate.get(k)
                setattr(g, k, None if t is None else t.data_ptr())
            g.use_rmsnorm = int(gate.get("use_rmsnorm", True))
            g.rms_eps = float(gate.get("rms_eps", 1e-5))
        return g

    @staticmethod
    def _scales(gate: dict, W_up, W_down) -> _Q8Scales:
        sc = _Q8Scales()
        if "W_g" in gate:
            sc.s_gate = gate["W_g"]["s"].data_ptr()
        else:
            sc.s_gate, sc.s_V = gate["U"]["s"].data_ptr(), gate["V"]["s"].data_ptr()
        sc.s_up, sc.s_down = W_up["s"].data_ptr(), W_down["s"].data_ptr()
        return sc

    def _stream(self, stream):
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        return ctypes.c_void_p(s.cuda_stream)

    def _call(self, fn, name, x, gate, b_g, W_up, W_down, act, y, stream):
        B = 1 if x.dim() == 1 else x.shape[0]
        g = self._gate(gate)
        self._keep = (x, gate, b_g, W_up, W_down, y)
        _check(name, fn(self._h, _ptr(x), B, ctypes.byref(g), _ptr(b_g), _ptr(W_up), _ptr(W_down),
                        ACT[act] if isinstance(act, str) else int(act), _ptr(y), self._stream(stream)))
        self._sync_check(name, B, gate)
        return y

    def status_words(self, n: int = 8):
        """The first ``n`` 32-bit words of the device status block (synchronises): [0] status, [1] length of the
        index list, [3] site + 256 * CTA of the last wait that gave up, [4] number of the last failed bounds check."""
        torch.cuda.synchronize(self.device)
        off = self._ws_ptr - self.workspace.data_ptr()
        return self.workspace[off:off + 4 * n].view(torch.int32).cpu().tolist()

    def _sync_check(self, name, B, gate):
        """With SFFN_SYNC_CHECK=1 in the environment every call is followed by a synchronisation and a look at the
        status word, so that the call that set it is the one that raises (diagnostics; slow)."""
        if os.environ.get("SFFN_SYNC_CHECK") != "1" or torch.cuda.is_current_stream_capturing():
            return
        w = self.status_words()
        if w[0] != 0:
            raise RuntimeError(f"{name} (B={B}, {'lopa' if 'V' in gate else 'standard'} gate, D={self.D}, H={self.H}): "
                               f"device status {w[0]}, site {w[3] % 256}, CTA {w[3] // 256}, words {w}")

    def _call_q8(self, fn, name, x, gate, b_g, W_up, W_down, act, y, stream):
        B = 1 if x.dim() == 1 else x.shape[0]
        g, sc = self._gate(gate), self._scales(gate, W_up, W_down)
        self._keep = (x, gate, b_g, W_up, W_down, y)
        _check(name, fn(self._h, _ptr(x), B, ctypes.byref(g), _ptr(b_g), _ptr(_codes(W_up)), _ptr(_codes(W_down)),
                        ctypes.byref(sc), ACT[act] if isinstance(act, str) else int(act), _ptr(y),
                        self._stream(stream)))
        return y

    def prepared(self, x, gate, b_g, W_up, W_down, act, y, *, dense=False, host=False, stream=None):
        """Marshals one call once and returns a zero-argument callable that issues it (for launch
        loops where per-call marshalling would dominate).  The stream is fixed at preparation."""
        B = 1 if x.dim() == 1 else x.shape[0]
        g = self._gate(gate)
        a = ACT[act] if isinstance(act, str) else int(act)
        if isinstance(W_up, dict):  # weight-only int8
            if host:
                raise ValueError("the host entry point takes fp32 / bf16 weights")
            if W_up["q"].dtype == torch.uint8:  # packed 4-bit codes
                fn = self.lib.dense_ffn_forward_q4 if dense else self.lib.sparse_ffn_forward_q4
            else:
                fn = self.lib.dense_ffn_forward_q8 if dense else self.lib.sparse_ffn_forward_q8
            sc = self._scales(gate, W_up, W_down)
            args = (self._h, _ptr(x), B, ctypes.byref(g), _ptr(b_g), _ptr(_codes(W_up)), _ptr(_codes(W_down)),
                    ctypes.byref(sc), a, _ptr(y), self._stream(stream))
            keep = (x, gate, b_g, W_up, W_down, y, g, sc)
        else:
            fn = (self.lib.sparse_ffn_forward_host if host else
                  self.lib.dense_ffn_forward if dense else self.lib.sparse_ffn_forward)
            args = (self._h, _ptr(x), B, ctypes.byref(g), _ptr(b_g), _ptr(W_up), _ptr(W_down), a, _ptr(y),
                    self._stream(stream))
            keep = (x, gate, b_g, W_up, W_down, y, g)

        def call(_fn=fn, _args=args, _keep=keep):
            rc = _fn(*_args)
            if rc:
                raise SFFNError("prepared call", rc)

        return call

    def sparse_ffn_forward(self, x, gate, b_g, W_up, W_down, act="relu", y=None, stream=None):
        """y = W_down^T (A(gate(x) + b_g) * (W_up x)) touching only the rows of fired neurons."""
        if y is None:
            y = torch.empty((*x.shape[:-1], self.D), dtype=torch.float32, device=x.device)
        return self._call(self.lib.sparse_ffn_forward, "sparse_ffn_forward", x, gate, b_g, W_up, W_down, act, y, stream)

    def dense_ffn_forward(self, x, gate, b_g, W_up, W_down, act="relu", y=None, stream=None):
        """The dense comparator: same function, all H rows read."""
        if y is None:
            y = torch.empty((*x.shape[:-1], self.D), dtype=torch.float32, device=x.device)
        return self._call(self.lib.dense_ffn_forward, "dense_ffn_forward", x, gate, b_g, W_up, W_down, act, y, stream)

    def sparse_ffn_forward_q8(self, x, gate, b_g, W_up, W_down, act="relu", y=None, stream=None):
        """:meth:`sparse_ffn_forward` on int8 weights with one fp32 scale per row (see the class docstring)."""
        if y is None:
            y = torch.empty((*x.shape[:-1], self.D), dtype=torch.float32, device=x.device)
        return self._call_q8(self.lib.sparse_ffn_forward_q8, "sparse_ffn_forward_q8", x, gate, b_g, W_up, W_down,
                             act, y, stream)

    def dense_ffn_forward_q8(self, x, gate, b_g, W_up, W_down, act="relu", y=None, stream=None):
        """The dense comparator on int8 weights."""
        if y is None:
            y = torch.empty((*x.shape[:-1], self.D), dtype=torch.float32, device=x.device)
        return self._call_q8(self.lib.dense_ffn_forward_q8, "dense_ffn_forward_q8", x, gate, b_g, W_up, W_down,
                             act, y, stream)

    def sparse_ffn_forward_q4(self, x, gate, b_g, W_up, W_down, act="relu", y=None, stream=None):
        """:meth:`sparse_ffn_forward` on 4-bit weights: every matrix is ``dict(q=uint8 [rows, cols / 2], s=float32
        [rows])``, two's-complement codes, even column in the low nibble (sparse_ffn_forward_q4 of the header)."""
        if y is None:
            y = torch.empty((*x.shape[:-1], self.D), dtype=torch.float32, device=x.device)
        return self._call_q8(self.lib.sparse_ffn_forward_q4, "sparse_ffn_forward_q4", x, gate, b_g, W_up, W_down,
                             act, y, stream)

    def dense_ffn_forward_q4(self, x, gate, b_g, W_up, W_down, act="relu", y=None, stream=None):
        """The dense comparator on 4-bit weights."""
        if y is None:
            y = torch.empty((*x.shape[:-1], self.D), dtype=torch.float32, device=x.device)
        return self._call_q8(self.lib.dense_ffn_forward_q4, "dense_ffn_forward_q4", x, gate, b_g, W_up, W_down,
                             act, y, stream)

    def sparse_ffn_forward_host(self, x_host, gate, b_g, W_up, W_down, act, y_host, stream=None):
        """End-to-end variant: x_host / y_host are (pinned) host tensors, weights on the device."""
        assert not x_host.is_cuda and not y_host.is_cuda
        return self._call(self.lib.sparse_ffn_forward_host, "sparse_ffn_forward_host", x_host, gate, b_g,
                          W_up, W_down, act, y_host, stream)

    def last_active(self, stream=None) -> torch.Tensor:
        """Ascending indices of the neurons that fired in the last sparse call (union for B > 1)."""
        idx, cnt = ctypes.c_void_p(), ctypes.c_void_p()
        _check("sffn_last_active", self.lib.sffn_last_active(self._h, ctypes.byref(idx), ctypes.byref(cnt),
                                                             self._stream(stream)))
        torch.cuda.synchronize(self.device)
        off_idx, off_cnt = idx.value - self.workspace.data_ptr(), cnt.value - self.workspace.data_ptr()
        n = int(self.workspace[off_cnt:off_cnt + 4].view(torch.int32).item())
        return self.workspace[off_idx:off_idx + 4 * n].view(torch.int32).clone()

    def device_status(self) -> int:
        out = ctypes.c_int(0)
        _check("sffn_last_device_status", self.lib.sffn_last_device_status(self._h, ctypes.byref(out)))
        return out.value

    def reset(self, stream=None):
        """Clears the device status word and the arrival counters after a device-side timeout."""
        _check("sffn_reset", self.lib.sffn_reset(self._h, self._stream(stream)))

    def launch_count(self) -> int:
        out = ctypes.c_longlong(0)
        _check("sffn_launch_count", self.lib.sffn_launch_count(self._h, ctypes.byref(out)))
        return out.value
