"""ctypes binding of libadacgd.so: the same entry points as include/adacgd.h.

torch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

TOPK, QUANT = 0, 1
PRED_LAZY, PRED_ABSOLUTE, PRED_RELATIVE, PRED_NEVER, PRED_ALWAYS = 0, 1, 2, 3, 4
LOSS_LOGISTIC_NCVX, LOSS_LOGISTIC_L2, LOSS_LEAST_SQUARES, LOSS_NONE = 0, 1, 2, 3
LAYOUT_DENSE, LAYOUT_CSR = 0, 1
FLAG_HOST_STAGING = 1
FLAG_INCREMENTAL_FORWARD = 2
STATE = dict(x=0, G=1, grad=2, gt=3, gm=4, step=5, bits_up=6, bits_down=7, levels=8, flags=9, rechecks=10, fallbacks=11, list_levels=12, device=13, inc_columns=14, refreshes=15)
STATUS = {0: "OK", 1: "INVALID_ARG", 2: "BAD_ORDER", 3: "NONFINITE", 4: "WORKSPACE", 5: "CUDA", 6: "UNSUPPORTED"}

EXPORTED_SYMBOLS = [
    "adacgd_workspace_bytes", "adacgd_init", "adacgd_step", "adacgd_compress", "adacgd_compress_host",
    "adacgd_gradient", "adacgd_get_state", "adacgd_set_state", "adacgd_last_error", "adacgd_destroy",
    "adacgd_launch_count", "adacgd_profile_kernel_count", "adacgd_profile_kernel_name", "adacgd_profile_enable",
    "adacgd_profile_read", "adacgd_compress_noalloc", "adacgd_message_bits", "adacgd_set_refresh_period",
]

Cand = Tuple[int, int]


class AdacgdError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"adacgd status {STATUS.get(status, status)}: {message}")
        self.status = status


class _Cand(C.Structure):
    _fields_ = [("kind", C.c_int32), ("reserved", C.c_int32), ("param", C.c_int64)]


class _Pred(C.Structure):
    _fields_ = [("kind", C.c_int32), ("param", C.c_float)]


class _Cset(C.Structure):
    _fields_ = [("cands", C.POINTER(_Cand)), ("m", C.c_int32), ("zeta", C.c_float), ("preds", C.POINTER(_Pred))]


class _Problem(C.Structure):
    _fields_ = [("loss", C.c_int32), ("lambda_", C.c_float), ("n", C.c_int32), ("layout", C.c_int32),
                ("d", C.c_int64), ("m_rows", C.c_int64), ("A", C.c_void_p), ("target", C.c_void_p),
                ("csr_rowptr", C.c_void_p), ("csr_col", C.c_void_p), ("csr_val", C.c_void_p), ("csr_nnz", C.c_int64)]


class StepReport(C.Structure):
    _fields_ = [("loss", C.c_double), ("bits_up", C.c_uint64), ("bits_down", C.c_uint64),
                ("master_level", C.c_int32), ("exact_rechecks", C.c_int32)]


_LIB = None


def library_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libadacgd.so")


def load_library():
    """Loads libadacgd.so; raises if it has not been built (there is no fallback)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -m paper_2211_00188_b200.build`")
    lib = C.CDLL(path)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    lib.adacgd_workspace_bytes.argtypes = [C.POINTER(_Problem), C.POINTER(_Cset), C.POINTER(_Cset), i32,
                                           C.POINTER(C.c_size_t)]
    lib.adacgd_init.argtypes = [C.POINTER(vp), C.POINTER(_Problem), C.POINTER(_Cset), C.POINTER(_Cset), vp,
                                C.c_float, i32, i32, vp, C.c_size_t, vp]
    lib.adacgd_step.argtypes = [vp, i32, C.POINTER(StepReport), C.POINTER(i32)]
    lib.adacgd_compress.argtypes = [vp, vp, vp, vp, i32, i64, C.POINTER(_Cset), vp, vp, vp, vp, vp, vp, i64, vp]
    lib.adacgd_compress_host.argtypes = [vp, vp, vp, vp, i32, i64, C.POINTER(_Cset), vp, vp, vp]
    lib.adacgd_gradient.argtypes = [vp, vp, vp, C.POINTER(C.c_double)]
    lib.adacgd_get_state.argtypes = [vp, i32, vp, C.c_size_t, i32]
    lib.adacgd_set_state.argtypes = [vp, i32, vp, C.c_size_t, i32]
    lib.adacgd_last_error.argtypes = [vp]
    lib.adacgd_last_error.restype = C.c_char_p
    lib.adacgd_destroy.argtypes = [vp]
    lib.adacgd_destroy.restype = None
    lib.adacgd_launch_count.argtypes = [vp]
    lib.adacgd_launch_count.restype = i64
    lib.adacgd_compress_noalloc.argtypes = [vp, vp, vp, i32, i64, C.POINTER(_Cset), vp, vp, vp, vp]
    lib.adacgd_set_refresh_period.argtypes = [vp, i32]
    lib.adacgd_message_bits.argtypes = [C.POINTER(_Cand), i64]
    lib.adacgd_message_bits.restype = C.c_uint64
    lib.adacgd_profile_kernel_count.argtypes = []
    lib.adacgd_profile_kernel_name.argtypes = [i32]
    lib.adacgd_profile_kernel_name.restype = C.c_char_p
    lib.adacgd_profile_enable.argtypes = [vp, i32]
    lib.adacgd_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i64)]
    for name in EXPORTED_SYMBOLS:
        if name not in ("adacgd_last_error", "adacgd_destroy", "adacgd_launch_count",
                        "adacgd_profile_kernel_name", "adacgd_message_bits"):
            getattr(lib, name).restype = i32
    _LIB = lib
    return lib


def _cset(cands: Optional[Sequence[Cand]], zeta: float, preds=None):
    """Returns (struct, keepalive).  preds: None, or one (kind, param) per level 0 .. m-1."""
    cands = list(cands or [])
    arr = (_Cand * max(1, len(cands)))()
    for i, (kind, param) in enumerate(cands):
        arr[i].kind, arr[i].reserved, arr[i].param = int(kind), 0, int(param)
    parr = None
    if preds is not None:
        if len(preds) != len(cands):
            raise ValueError("one trigger per level 0 .. m-1: len(preds) must equal len(cands)")
        parr = (_Pred * max(1, len(preds)))()
        for i, (kind, param) in enumerate(preds):
            parr[i].kind, parr[i].param = int(kind), float(param)
    cs = _Cset(C.cast(arr, C.POINTER(_Cand)), len(cands), float(zeta),
               C.cast(parr, C.POINTER(_Pred)) if parr is not None else None)
    return cs, (arr, parr)


def message_bits(cand: Cand, d: int) -> int:
    """adacgd_message_bits: bits of the message a worker sends with candidate `cand` at dimension d."""
    c = _Cand(int(cand[0]), 0, int(cand[1]))
    return int(load_library().adacgd_message_bits(C.byref(c), int(d)))


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


class AdaCGD:
    """Owns a context and the device workspace behind it.  Methods mirror the C entry points."""

    def __init__(self, n: int, d: int, worker: Sequence[Cand] = (), worker_zeta: float = 0.0,
                 master: Sequence[Cand] = (), master_zeta: float = 0.0, *, loss: int = LOSS_NONE,
                 lam: float = 0.0, A=None, target=None, csr=None, x0=None, gamma: float = 1.0, g0_mode: int = 1,
                 host_staging: bool = False, incremental_forward: bool = False, worker_preds=None, master_preds=None,
                 device="cuda:0", stream=None):
        import torch

        self.torch = torch
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("adacgd needs a CUDA device; there is no CPU path")
        self.device = torch.device(device)
        self.n, self.d = int(n), int(d)
        self.worker, self.worker_zeta = list(worker), float(worker_zeta)
        self.master, self.master_zeta = list(master), float(master_zeta)
        self._keep = [A, target, x0, csr]
        m_rows = 0
        layout, rowptr, col, val, nnz = LAYOUT_DENSE, None, None, None, 0
        if loss != LOSS_NONE:
            assert target.dtype == torch.float32 and target.is_contiguous() and target.is_cuda
            m_rows = target.shape[1]
            assert tuple(target.shape) == (n, m_rows)
            if csr is not None:   # (rowptr int64 [n*m+1], col int32 [nnz], val float32 [nnz]) on the device
                layout = LAYOUT_CSR
                rowptr, col, val = csr
                assert rowptr.dtype == torch.int64 and col.dtype == torch.int32 and val.dtype == torch.float32
                assert rowptr.numel() == n * m_rows + 1 and col.numel() == val.numel()
                assert rowptr.is_cuda and col.is_cuda and val.is_cuda
                nnz = col.numel()
            else:
                assert A.dtype == torch.float32 and A.is_contiguous() and A.is_cuda
                assert tuple(A.shape) == (n, m_rows, d)
        self.problem = _Problem(loss, float(lam), self.n, layout, self.d, m_rows, _ptr(A) if A is not None else None,
                                _ptr(target) if target is not None else None, _ptr(rowptr), _ptr(col), _ptr(val), nnz)
        self.flags = (FLAG_HOST_STAGING if host_staging else 0) | (FLAG_INCREMENTAL_FORWARD if incremental_forward else 0)
        self.worker_preds, self.master_preds = worker_preds, master_preds
        wcs, k1 = _cset(self.worker, worker_zeta, worker_preds)
        mcs, k2 = _cset(self.master, master_zeta, master_preds)
        nbytes = C.c_size_t(0)
        self._check(self.lib.adacgd_workspace_bytes(C.byref(self.problem), C.byref(wcs), C.byref(mcs), self.flags,
                                                    C.byref(nbytes)), None)
        self.workspace = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        ctx = C.c_void_p()
        self._check(self.lib.adacgd_init(C.byref(ctx), C.byref(self.problem), C.byref(wcs), C.byref(mcs),
                                         _ptr(x0) if x0 is not None else None, float(gamma), int(g0_mode), self.flags,
                                         C.c_void_p(base), nbytes.value, C.c_void_p(self.stream.cuda_stream)), None)
        self.ctx = ctx
        self.workspace_bytes = nbytes.value

    # -- helpers ---------------------------------------------------------
    def _check(self, status: int, ctx):
        if status != 0:
            msg = self.lib.adacgd_last_error(ctx)
            raise AdacgdError(status, msg.decode() if msg else "")

    def close(self):
        if getattr(self, "ctx", None):
            self.lib.adacgd_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- entry points ------------------------------------------------------
    def compress(self, X, G, Y, cands: Optional[Sequence[Cand]] = None, zeta: Optional[float] = None, *,
                 mean_out=None, level=None, bits=None, err=None, D=None, kept_idx=None, kept_cnt=None, preds=None):
        """adacgd_compress on device tensors; G is updated in place."""
        rows, d = X.shape
        if cands is None and preds is None:
            preds = self.worker_preds
        cs, keep = _cset(self.worker if cands is None else cands, self.worker_zeta if zeta is None else zeta, preds)
        stride = kept_idx.shape[1] if kept_idx is not None else 0
        self._check(self.lib.adacgd_compress(self.ctx, _ptr(X), _ptr(G), _ptr(Y), rows, d, C.byref(cs), _ptr(mean_out),
                                             _ptr(level), _ptr(bits), _ptr(err), _ptr(D), _ptr(kept_idx), stride,
                                             _ptr(kept_cnt)), self.ctx)

    def compress_host(self, X, G, Y, cands=None, zeta=None, *, mean_out=None, level=None, bits=None):
        """adacgd_compress_host on host (preferably pinned) tensors; G is updated in place."""
        rows, d = X.shape
        cs, keep = _cset(self.worker if cands is None else cands, self.worker_zeta if zeta is None else zeta)
        self._check(self.lib.adacgd_compress_host(self.ctx, _ptr(X), _ptr(G), _ptr(Y), rows, d, C.byref(cs),
                                                  _ptr(mean_out), _ptr(level), _ptr(bits)), self.ctx)

    def gradient(self, x, out, want_loss: bool = False):
        loss = C.c_double(0.0)
        self._check(self.lib.adacgd_gradient(self.ctx, _ptr(x), _ptr(out), C.byref(loss) if want_loss else None),
                    self.ctx)
        return loss.value if want_loss else None

    def step(self, n_steps: int = 1, report: bool = False):
        """adacgd_step; with report=True returns (list of dict, levels [n_steps][n])."""
        if not report:
            self._check(self.lib.adacgd_step(self.ctx, n_steps, None, None), self.ctx)
            return None
        rep = (StepReport * n_steps)()
        lev = (C.c_int32 * (n_steps * self.n))()
        self._check(self.lib.adacgd_step(self.ctx, n_steps, rep, lev), self.ctx)
        recs = [dict(loss=r.loss, bits_up=r.bits_up, bits_down=r.bits_down, master_level=r.master_level,
                     exact_rechecks=r.exact_rechecks) for r in rep]
        levels = [list(lev[t * self.n:(t + 1) * self.n]) for t in range(n_steps)]
        return recs, levels

    def get_state(self, which: str):
        torch = self.torch
        n, d = self.n, self.d
        shapes = dict(x=((d,), torch.float32), G=((n, d), torch.float32), grad=((n, d), torch.float32),
                      gt=((d,), torch.float32), gm=((d,), torch.float32), levels=((n,), torch.int32))
        if which in shapes:
            shape, dt = shapes[which]
            out = torch.empty(shape, dtype=dt, device=self.device)
            self._check(self.lib.adacgd_get_state(self.ctx, STATE[which], _ptr(out), out.numel() * out.element_size(), 1),
                        self.ctx)
            return out
        buf = C.c_uint64(0) if which not in ("flags", "rechecks", "fallbacks", "list_levels", "device") else C.c_uint32(0)
        self._check(self.lib.adacgd_get_state(self.ctx, STATE[which], C.byref(buf), C.sizeof(buf), 0), self.ctx)
        return int(buf.value)

    def set_state(self, which: str, value):
        torch = self.torch
        if which in ("x", "G", "grad", "gt", "gm"):
            t = value.to(device=self.device, dtype=torch.float32).contiguous()
            self._check(self.lib.adacgd_set_state(self.ctx, STATE[which], _ptr(t), t.numel() * 4, 1), self.ctx)
        else:
            buf = C.c_uint64(int(value))
            self._check(self.lib.adacgd_set_state(self.ctx, STATE[which], C.byref(buf), 8, 0), self.ctx)

    def set_refresh_period(self, period: int):
        """adacgd_set_refresh_period: iterations between full recomputations of the kept forward products."""
        self._check(self.lib.adacgd_set_refresh_period(self.ctx, int(period)), self.ctx)

    def profile_enable(self, max_records: int):
        self._check(self.lib.adacgd_profile_enable(self.ctx, int(max_records)), self.ctx)

    def profile_read(self):
        """Returns {kernel name: (total ms, timed launches)} and clears the records."""
        k = self.lib.adacgd_profile_kernel_count()
        ms = (C.c_double * k)()
        cnt = (C.c_int64 * k)()
        self._check(self.lib.adacgd_profile_read(self.ctx, ms, cnt), self.ctx)
        return {self.lib.adacgd_profile_kernel_name(i).decode(): (ms[i], int(cnt[i])) for i in range(k) if cnt[i]}

    def launch_count(self) -> int:
        return int(self.lib.adacgd_launch_count(self.ctx))


NOALLOC_MAX_ROWS = 4
NOALLOC_MAX_D = 4194304


def compress_noalloc(X, G, Y, cands: Sequence[Cand], zeta: float, *, mean_out=None, level=None, bits=None,
                     stream=None):
    """adacgd_compress_noalloc on device tensors: the same result as AdaCGD.compress for
    callers that may not allocate device memory.  Needs no context and no workspace (the
    library's built-in 2 MiB scratch is used), accepts at most NOALLOC_MAX_ROWS rows of at
    most NOALLOC_MAX_D columns, enqueues on `stream` (default: torch's current stream) and
    must not run concurrently with another call on the same GPU."""
    import torch

    lib = load_library()
    rows, d = X.shape
    cs, keep = _cset(cands, zeta)
    st = stream if stream is not None else torch.cuda.current_stream(X.device)
    with torch.cuda.device(X.device):
        status = lib.adacgd_compress_noalloc(_ptr(X), _ptr(G), _ptr(Y), rows, d, C.byref(cs), _ptr(mean_out),
                                             _ptr(level), _ptr(bits), C.c_void_p(st.cuda_stream))
    if status != 0:
        raise AdacgdError(status, lib.adacgd_last_error(None).decode())
