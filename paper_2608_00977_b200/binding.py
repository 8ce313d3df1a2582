"""Thin ctypes layer over libtsid.so: argument marshalling only.

Names and arguments follow include/tsid.h.  Device memory and streams come from
PyTorch tensors (``.data_ptr()``); every step of the path runs in the library's
kernels.  A missing library is an error: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtsid.so")

TSID_OK = 0
STATUS_NAMES = ["TSID_OK", "TSID_ERR_INVALID_ARG", "TSID_ERR_INDEX_RANGE", "TSID_ERR_DUPLICATE",
                "TSID_ERR_UNSORTED", "TSID_ERR_OOM", "TSID_ERR_CUDA", "TSID_ERR_UNSUPPORTED",
                "TSID_ERR_NONFINITE", "TSID_ERR_TOO_LARGE"]
TSID_ERR_TOO_LARGE = 9
(TSID_ERR_INVALID_ARG, TSID_ERR_INDEX_RANGE, TSID_ERR_DUPLICATE, TSID_ERR_UNSORTED, TSID_ERR_OOM,
 TSID_ERR_CUDA, TSID_ERR_UNSUPPORTED, TSID_ERR_NONFINITE) = range(1, 9)
TSID_F32, TSID_BF16_SHADOW = 0, 1
TSID_PATH_AUTO, TSID_PATH_SPARSE, TSID_PATH_DENSE_TC, TSID_PATH_HYBRID = 0, 1, 2, 3
TSID_CLIP_NONE, TSID_CLIP_ASYM_STEP, TSID_CLIP_ASYM_GRAD, TSID_CLIP_ASYM_ENTRY = 0, 1, 2, 3
TSID_NORM_NONE, TSID_NORM_COUNT = 0, 1
TSID_VALIDATE, TSID_INPUT_ROW_SORTED, TSID_VALUES_U8 = 1, 2, 4

# every symbol include/tsid.h declares
EXPORTS = ["tsid_workspace_bytes", "tsid_template_create", "tsid_grad_step", "tsid_fit", "tsid_loss",
           "tsid_check", "tsid_destroy", "tsid_get_layout", "tsid_residuals", "tsid_get_info",
           "tsid_last_error", "tsid_workspace_bytes_host", "tsid_fit_host", "tsid_set_profiling",
           "tsid_get_pass_times", "tsid_sse_noalloc", "tsid_sample_workspace_bytes", "tsid_sample_template",
           "tsid_extend_workspace_bytes", "tsid_extend", "tsid_grad", "tsid_apply", "tsid_get_counts",
           "tsid_set_norm_counts", "tsid_apply_sliced", "tsid_get_hybrid_info", "tsid_get_step_times",
           "tsid_get_fit_launches",
           "tsid_debug_stall_tile_pass", "tsid_workspace_bytes_batched", "tsid_template_create_batched",
           "tsid_grad_step_batch"]


class TsidConfig(C.Structure):
    _fields_ = [("m", C.c_int32), ("n", C.c_int32), ("k", C.c_int32), ("nnz", C.c_int64),
                ("precision", C.c_int32), ("path", C.c_int32),
                ("eta", C.c_float), ("lam", C.c_float), ("xi", C.c_float),
                ("clip", C.c_int32), ("norm_p", C.c_int32), ("norm_q", C.c_int32),
                ("flags", C.c_uint32), ("stream", C.c_void_p), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_size_t)]


class TsidExtendConfig(C.Structure):
    _fields_ = [("m", C.c_int32), ("d", C.c_int32), ("k", C.c_int32), ("n_cols", C.c_int32),
                ("chunk_cols", C.c_int32), ("iters", C.c_int32),
                ("eta", C.c_float), ("lam", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("flags", C.c_uint32), ("stream", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


class TsidError(RuntimeError):
    def __init__(self, status, message):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__("%s: %s" % (name, message))


_lib = None


def lib():
    """Loads libtsid.so (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libtsid.so is missing: run `python -c 'import __graft_entry__ as g; g.build()'` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp = C.c_void_p
        L.tsid_workspace_bytes.argtypes = [C.POINTER(TsidConfig), C.POINTER(C.c_size_t)]
        L.tsid_template_create.argtypes = [C.POINTER(TsidConfig), vp, vp, vp, C.POINTER(vp)]
        L.tsid_grad_step.argtypes = [vp, vp, vp, vp, vp]
        L.tsid_fit.argtypes = [vp, vp, vp, C.c_int32, C.c_int32, C.POINTER(C.c_double)]
        L.tsid_grad.argtypes = [vp, vp, vp, vp, vp]
        L.tsid_apply.argtypes = [vp, vp, vp, vp, vp]
        L.tsid_get_counts.argtypes = [vp, vp, vp]
        L.tsid_set_norm_counts.argtypes = [vp, vp, vp]
        L.tsid_apply_sliced.argtypes = [vp, vp, vp, C.POINTER(vp), C.POINTER(vp), C.c_int32, C.c_int32]
        L.tsid_loss.argtypes = [vp, vp, vp, C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.tsid_check.argtypes = [vp]
        L.tsid_destroy.argtypes = [vp]
        L.tsid_get_layout.argtypes = [vp] + [C.POINTER(vp)] * 7
        L.tsid_residuals.argtypes = [vp, vp, vp, vp]
        L.tsid_get_info.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.tsid_get_fit_launches.argtypes = [vp, C.c_int32, C.POINTER(C.c_int64)]
        L.tsid_last_error.argtypes = [vp]
        L.tsid_get_hybrid_info.argtypes = [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
        L.tsid_workspace_bytes_host.argtypes = [C.POINTER(TsidConfig), C.POINTER(C.c_size_t)]
        L.tsid_fit_host.argtypes = [C.POINTER(TsidConfig), vp, vp, vp, vp, vp, C.c_int32, C.POINTER(C.c_double)]
        L.tsid_set_profiling.argtypes = [vp, C.c_int32]
        L.tsid_get_pass_times.argtypes = [vp, C.POINTER(C.c_int32)] + [C.POINTER(C.c_float)] * 3
        L.tsid_debug_stall_tile_pass.argtypes = [vp, C.c_int64, C.c_int32]
        L.tsid_workspace_bytes_batched.argtypes = [C.POINTER(TsidConfig), C.c_int32, C.POINTER(C.c_size_t)]
        L.tsid_template_create_batched.argtypes = [C.POINTER(TsidConfig), vp, vp, vp, vp, C.c_int32, C.POINTER(vp)]
        L.tsid_grad_step_batch.argtypes = [vp, C.c_int32, vp, vp, vp, vp]
        L.tsid_get_step_times.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_float)]
        L.tsid_sse_noalloc.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int64, vp, vp, vp, vp, vp, vp, vp]
        L.tsid_sample_workspace_bytes.argtypes = [C.c_int32, C.c_int64, C.POINTER(C.c_size_t)]
        L.tsid_sample_template.argtypes = [C.c_int32, C.c_int32, C.c_int64, C.c_double, C.c_uint64, vp, vp, vp, vp, vp,
                                           C.c_size_t, vp, vp, vp, vp, C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
        L.tsid_extend_workspace_bytes.argtypes = [C.POINTER(TsidExtendConfig), vp, C.POINTER(C.c_size_t)]
        L.tsid_extend.argtypes = [C.POINTER(TsidExtendConfig), vp, vp, vp, vp, vp, vp, C.POINTER(C.c_double)]
        L.tsid_last_error.restype = C.c_char_p
        for name in EXPORTS:
            if name != "tsid_last_error":
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _check_tensor(t, dtype, numel, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()
            and t.numel() == numel):
        raise ValueError("%s must be a contiguous CUDA tensor of %s with %d elements" % (name, dtype, numel))


def make_config(m, n, k, nnz, precision=TSID_F32, path=TSID_PATH_AUTO, eta=0.01, lam=0.0, xi=0.1,
                clip=TSID_CLIP_NONE, norm_p=TSID_NORM_NONE, norm_q=TSID_NORM_NONE, flags=0) -> TsidConfig:
    return TsidConfig(m, n, k, nnz, precision, path, eta, lam, xi, clip, norm_p, norm_q, flags, None, None, 0)


def tsid_workspace_bytes(cfg: TsidConfig) -> int:
    out = C.c_size_t(0)
    st = lib().tsid_workspace_bytes(C.byref(cfg), C.byref(out))
    if st != TSID_OK:
        raise TsidError(st, lib().tsid_last_error(None).decode())
    return out.value


class Template:
    """Owns the workspace tensor and the handle of one template (tsid_template_create ... tsid_destroy)."""

    def __init__(self, cfg: TsidConfig, rows: torch.Tensor, cols: torch.Tensor, vals: torch.Tensor,
                 stream: torch.cuda.Stream | None = None, batch: torch.Tensor | None = None, n_batches: int = 0):
        """batch / n_batches given: a mini-batch template (tsid_template_create_batched), stepped with
        tsid_grad_step_batch."""
        L = lib()
        nnz = int(cfg.nnz)
        if batch is not None:
            _check_tensor(batch, torch.int32, nnz, "batch")
        _check_tensor(rows, torch.int32, nnz, "rows")
        _check_tensor(cols, torch.int32, nnz, "cols")
        _check_tensor(vals, torch.float32, nnz, "vals")
        self.device = rows.device
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        if batch is None:
            need = tsid_workspace_bytes(cfg)
        else:
            out = C.c_size_t(0)
            st = L.tsid_workspace_bytes_batched(C.byref(cfg), int(n_batches), C.byref(out))
            if st != TSID_OK:
                raise TsidError(st, L.tsid_last_error(None).decode())
            need = out.value
        self.n_batches = int(n_batches) if batch is not None else 0
        self.workspace = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) & ~255
        self.cfg = TsidConfig.from_buffer_copy(cfg)
        self.cfg.stream = self.stream.cuda_stream
        self.cfg.workspace = base
        self.cfg.workspace_bytes = need
        self.m, self.n, self.k, self.nnz = int(cfg.m), int(cfg.n), int(cfg.k), nnz
        h = C.c_void_p(None)
        with torch.cuda.device(self.device):
            if batch is None:
                st = L.tsid_template_create(C.byref(self.cfg), rows.data_ptr(), cols.data_ptr(), vals.data_ptr(),
                                            C.byref(h))
            else:
                st = L.tsid_template_create_batched(C.byref(self.cfg), rows.data_ptr(), cols.data_ptr(), vals.data_ptr(),
                                                    batch.data_ptr(), int(n_batches), C.byref(h))
        if st != TSID_OK:
            self.h = None
            raise TsidError(st, L.tsid_last_error(None).decode())
        self.h = h

    # -- the entry points, same names as the header ------------------------------------------------
    def _raise(self, st):
        raise TsidError(st, lib().tsid_last_error(self.h).decode())

    def _factors(self, P, Q):
        _check_tensor(P, torch.float32, self.m * self.k, "P")
        _check_tensor(Q, torch.float32, self.n * self.k, "Q")

    def tsid_grad_step(self, P, Q, gradP=None, gradQ=None):
        self._factors(P, Q)
        if gradP is not None:
            _check_tensor(gradP, torch.float32, self.m * self.k, "gradP")
        if gradQ is not None:
            _check_tensor(gradQ, torch.float32, self.n * self.k, "gradQ")
        st = lib().tsid_grad_step(self.h, P.data_ptr(), Q.data_ptr(),
                                  gradP.data_ptr() if gradP is not None else None,
                                  gradQ.data_ptr() if gradQ is not None else None)
        if st != TSID_OK:
            self._raise(st)

    def tsid_grad_step_batch(self, batch, P, Q, gradP=None, gradQ=None):
        self._factors(P, Q)
        st = lib().tsid_grad_step_batch(self.h, int(batch), P.data_ptr(), Q.data_ptr(),
                                        gradP.data_ptr() if gradP is not None else None,
                                        gradQ.data_ptr() if gradQ is not None else None)
        if st != TSID_OK:
            self._raise(st)

    def tsid_grad(self, P, Q, gradP, gradQ):
        self._factors(P, Q)
        _check_tensor(gradP, torch.float32, self.m * self.k, "gradP")
        _check_tensor(gradQ, torch.float32, self.n * self.k, "gradQ")
        st = lib().tsid_grad(self.h, P.data_ptr(), Q.data_ptr(), gradP.data_ptr(), gradQ.data_ptr())
        if st != TSID_OK:
            self._raise(st)

    def tsid_apply(self, P, Q, gradP, gradQ):
        self._factors(P, Q)
        _check_tensor(gradP, torch.float32, self.m * self.k, "gradP")
        _check_tensor(gradQ, torch.float32, self.n * self.k, "gradQ")
        st = lib().tsid_apply(self.h, P.data_ptr(), Q.data_ptr(), gradP.data_ptr(), gradQ.data_ptr())
        if st != TSID_OK:
            self._raise(st)

    def tsid_apply_sliced(self, P, gradP, q_ptrs, gq_ptrs, rank):
        """q_ptrs / gq_ptrs: device addresses (ints) of every rank's Q replica and partial G_Q."""
        _check_tensor(P, torch.float32, self.m * self.k, "P")
        _check_tensor(gradP, torch.float32, self.m * self.k, "gradP")
        world = len(q_ptrs)
        if len(gq_ptrs) != world:
            raise ValueError("q_ptrs and gq_ptrs must have one entry per rank")
        qa = (C.c_void_p * world)(*[int(x) for x in q_ptrs])
        ga = (C.c_void_p * world)(*[int(x) for x in gq_ptrs])
        st = lib().tsid_apply_sliced(self.h, P.data_ptr(), gradP.data_ptr(), qa, ga, int(rank), world)
        if st != TSID_OK:
            self._raise(st)

    def tsid_get_counts(self):
        cp = torch.empty(self.m, dtype=torch.int32, device=self.device)
        cq = torch.empty(self.n, dtype=torch.int32, device=self.device)
        st = lib().tsid_get_counts(self.h, cp.data_ptr(), cq.data_ptr())
        if st != TSID_OK:
            self._raise(st)
        return cp, cq

    def tsid_set_norm_counts(self, cnt_p=None, cnt_q=None):
        if cnt_p is not None:
            _check_tensor(cnt_p, torch.int32, self.m, "cnt_p")
        if cnt_q is not None:
            _check_tensor(cnt_q, torch.int32, self.n, "cnt_q")
        st = lib().tsid_set_norm_counts(self.h, cnt_p.data_ptr() if cnt_p is not None else None,
                                        cnt_q.data_ptr() if cnt_q is not None else None)
        if st != TSID_OK:
            self._raise(st)

    def tsid_fit(self, P, Q, epochs, loss_every=0):
        self._factors(P, Q)
        hist = None
        if loss_every > 0:
            hist = (C.c_double * (1 + epochs // loss_every))()
        st = lib().tsid_fit(self.h, P.data_ptr(), Q.data_ptr(), epochs, loss_every, hist)
        if st != TSID_OK:
            self._raise(st)
        return list(hist) if hist is not None else None

    def tsid_loss(self, P, Q):
        self._factors(P, Q)
        sse, obj = C.c_double(0), C.c_double(0)
        st = lib().tsid_loss(self.h, P.data_ptr(), Q.data_ptr(), C.byref(sse), C.byref(obj))
        if st != TSID_OK:
            self._raise(st)
        return sse.value, obj.value

    def tsid_check(self):
        st = lib().tsid_check(self.h)
        if st != TSID_OK:
            self._raise(st)

    def tsid_residuals(self, P, Q, e=None):
        self._factors(P, Q)
        if e is None:
            e = torch.empty(self.nnz, dtype=torch.float32, device=self.device)
        _check_tensor(e, torch.float32, self.nnz, "e")
        st = lib().tsid_residuals(self.h, P.data_ptr(), Q.data_ptr(), e.data_ptr())
        if st != TSID_OK:
            self._raise(st)
        return e

    def tsid_get_info(self):
        p, l = C.c_int32(0), C.c_int32(0)
        lib().tsid_get_info(self.h, C.byref(p), C.byref(l))
        return p.value, l.value

    def tsid_get_fit_launches(self, epochs):
        n = C.c_int64(0)
        st = lib().tsid_get_fit_launches(self.h, int(epochs), C.byref(n))
        if st != TSID_OK:
            self._raise(st)
        return n.value

    def tsid_get_hybrid_info(self):
        """(stored tiles, smallest entry count of a stored tile, entries left to the gather-reduce passes)."""
        a, b, c = C.c_int64(0), C.c_int32(0), C.c_int64(0)
        lib().tsid_get_hybrid_info(self.h, C.byref(a), C.byref(b), C.byref(c))
        return a.value, b.value, c.value

    def tsid_debug_stall_tile_pass(self, wait_cycles, item):
        st = lib().tsid_debug_stall_tile_pass(self.h, int(wait_cycles), int(item))
        if st != TSID_OK:
            self._raise(st)

    def tsid_set_profiling(self, enable):
        st = lib().tsid_set_profiling(self.h, int(enable))
        if st != TSID_OK:
            self._raise(st)

    def tsid_get_pass_times(self):
        """(steps, row_ms, col_ms, update_ms) summed over the recorded steps."""
        n = C.c_int32(0)
        a, b, c = C.c_float(0), C.c_float(0), C.c_float(0)
        st = lib().tsid_get_pass_times(self.h, C.byref(n), C.byref(a), C.byref(b), C.byref(c))
        if st != TSID_OK:
            self._raise(st)
        return n.value, a.value, b.value, c.value

    def tsid_get_step_times(self):
        """(steps, row_ms, col_ms, update_ms, tiles_ms) summed over the recorded steps."""
        n = C.c_int32(0)
        ms = (C.c_float * 4)()
        st = lib().tsid_get_step_times(self.h, C.byref(n), ms)
        if st != TSID_OK:
            self._raise(st)
        return n.value, ms[0], ms[1], ms[2], ms[3]

    def tsid_get_layout(self, copy=True):
        """The layout arrays as torch tensors (row_ptr, col_idx, val_csr, col_ptr, row_idx, val_csc, perm):
        copies, or with copy=False views into the workspace that die with the template."""
        ptrs = [C.c_void_p(None) for _ in range(7)]
        st = lib().tsid_get_layout(self.h, *[C.byref(p) for p in ptrs])
        if st != TSID_OK:
            self._raise(st)
        base = (self.workspace.data_ptr() + 255) & ~255
        spec = [(torch.int64, self.m + 1), (torch.int32, self.nnz), (torch.float32, self.nnz),
                (torch.int64, self.n + 1), (torch.int32, self.nnz), (torch.float32, self.nnz),
                (torch.int32, self.nnz)]   # perm is uint32; viewed as int32 (nnz < 2^31)
        out = []
        self.stream.synchronize()
        for p, (dt, cnt) in zip(ptrs, spec):
            off = p.value - base + (base - self.workspace.data_ptr())
            nbytes = cnt * torch.empty(0, dtype=dt).element_size()
            v = self.workspace[off:off + nbytes].view(dt)
            out.append(v.clone() if copy else v)
        return out

    def tsid_destroy(self):
        if getattr(self, "h", None) is not None:
            lib().tsid_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.tsid_destroy()
        except Exception:
            pass


def tsid_workspace_bytes_host(cfg: TsidConfig) -> int:
    out = C.c_size_t(0)
    st = lib().tsid_workspace_bytes_host(C.byref(cfg), C.byref(out))
    if st != TSID_OK:
        raise TsidError(st, lib().tsid_last_error(None).decode())
    return out.value


def tsid_fit_host(cfg: TsidConfig, rows, cols, vals, P, Q, epochs, workspace: torch.Tensor,
                  stream=None, want_sse=False):
    """Host-buffer call: rows/cols/vals/P/Q are CPU tensors (pinned for asynchronous copies); P, Q are
    overwritten with the fitted factors.  `workspace` is a CUDA uint8 tensor of at least
    tsid_workspace_bytes_host(cfg) + 256 bytes.  Returns the SSE if requested."""
    for t, dt, nm in ((rows, torch.int32, "rows"), (cols, torch.int32, "cols"), (vals, torch.float32, "vals"),
                      (P, torch.float32, "P"), (Q, torch.float32, "Q")):
        if t.is_cuda or t.dtype != dt or not t.is_contiguous():
            raise ValueError("%s must be a contiguous CPU tensor of %s" % (nm, dt))
    need = tsid_workspace_bytes_host(cfg)
    base = (workspace.data_ptr() + 255) & ~255
    if workspace.numel() - (base - workspace.data_ptr()) < need:
        raise ValueError("workspace too small: need %d bytes" % need)
    c = TsidConfig.from_buffer_copy(cfg)
    stream = stream if stream is not None else torch.cuda.current_stream(workspace.device)
    c.stream = stream.cuda_stream
    c.workspace = base
    c.workspace_bytes = need
    sse = C.c_double(0)
    with torch.cuda.device(workspace.device):
        st = lib().tsid_fit_host(C.byref(c), rows.data_ptr(), cols.data_ptr(), vals.data_ptr(), P.data_ptr(),
                                 Q.data_ptr(), int(epochs), C.byref(sse) if want_sse else None)
    if st != TSID_OK:
        raise TsidError(st, lib().tsid_last_error(None).decode())
    return sse.value if want_sse else None


def tsid_sse_noalloc(m, n, k, rows, cols, vals, P, Q, out, stream=None):
    """SSE of a COO template without a handle or workspace: `out` (CUDA float64 tensor with one element)
    receives the result asynchronously on `stream`.  For callers that may not allocate device memory: this
    wrapper allocates nothing either (all tensors, the output included, come from the caller)."""
    nnz = int(rows.numel())
    _check_tensor(rows, torch.int32, nnz, "rows")
    _check_tensor(cols, torch.int32, nnz, "cols")
    _check_tensor(vals, torch.float32, nnz, "vals")
    _check_tensor(P, torch.float32, m * k, "P")
    _check_tensor(Q, torch.float32, n * k, "Q")
    _check_tensor(out, torch.float64, 1, "out")
    stream = stream if stream is not None else torch.cuda.current_stream(P.device)
    with torch.cuda.device(P.device):
        st = lib().tsid_sse_noalloc(m, n, k, nnz, rows.data_ptr(), cols.data_ptr(), vals.data_ptr(), P.data_ptr(),
                                    Q.data_ptr(), stream.cuda_stream, out.data_ptr())
    if st != TSID_OK:
        raise TsidError(st, "tsid_sse_noalloc refused or failed")


def tsid_sample_template(m, n, rows, cols, vals, alpha, seed, stream=None):
    """Column sampling + template extraction.  Returns (colmap int32[n], rows', cols', vals', d) as CUDA
    tensors (the triples trimmed to the number of template entries)."""
    nnz = int(rows.numel())
    _check_tensor(rows, torch.int32, nnz, "rows")
    _check_tensor(cols, torch.int32, nnz, "cols")
    _check_tensor(vals, torch.float32, nnz, "vals")
    dev = rows.device
    need = C.c_size_t(0)
    st = lib().tsid_sample_workspace_bytes(n, nnz, C.byref(need))
    if st != TSID_OK:
        raise TsidError(st, "tsid_sample_workspace_bytes")
    ws = torch.empty(need.value + 256, dtype=torch.uint8, device=dev)
    base = (ws.data_ptr() + 255) & ~255
    colmap = torch.empty(n, dtype=torch.int32, device=dev)
    ro, co = torch.empty(max(nnz, 1), dtype=torch.int32, device=dev), torch.empty(max(nnz, 1), dtype=torch.int32, device=dev)
    vo = torch.empty(max(nnz, 1), dtype=torch.float32, device=dev)
    d, kept = C.c_int32(0), C.c_int64(0)
    stream = stream if stream is not None else torch.cuda.current_stream(dev)
    with torch.cuda.device(dev):
        st = lib().tsid_sample_template(m, n, nnz, float(alpha), int(seed), rows.data_ptr(), cols.data_ptr(),
                                        vals.data_ptr(), stream.cuda_stream, base, need.value, colmap.data_ptr(),
                                        ro.data_ptr(), co.data_ptr(), vo.data_ptr(), C.byref(d), C.byref(kept))
    if st != TSID_OK:
        raise TsidError(st, "tsid_sample_template")
    k = kept.value
    return colmap, ro[:k], co[:k], vo[:k], d.value


TSID_EXTEND_COLD_START, TSID_EXTEND_TC = 1, 2


def tsid_extend(P, Q, col_ptr, row_idx, vals, C0, chunk_cols, iters, eta, lam, beta1=0.9, beta2=0.999, eps=1e-8,
                want_sse=False, stream=None, cold_start=False, tensor_cores=False):
    """Stage II extension.  P (m x k), Q (d x k): CUDA fp32 tensors.  col_ptr (int64), row_idx (int32),
    vals (fp32), C0 (fp32 [n_cols, d]): CPU tensors (pinned for asynchronous copies); C0 is overwritten with
    the fitted coefficients.  Returns the SSE if requested."""
    m, k = P.shape
    d = Q.shape[0]
    n_cols = col_ptr.numel() - 1
    for t, dt in ((col_ptr, torch.int64), (row_idx, torch.int32), (vals, torch.float32), (C0, torch.float32)):
        if t.is_cuda or t.dtype != dt or not t.is_contiguous():
            raise ValueError("host tensors must be contiguous CPU tensors of the documented dtypes")
    _check_tensor(P, torch.float32, m * k, "P")
    _check_tensor(Q, torch.float32, d * k, "Q")
    if C0.numel() != n_cols * d:
        raise ValueError("C0 must have n_cols * d elements")
    dev = P.device
    stream = stream if stream is not None else torch.cuda.current_stream(dev)
    cfg = TsidExtendConfig(m, d, k, n_cols, chunk_cols, iters, eta, lam, beta1, beta2, eps,
                           (TSID_EXTEND_COLD_START if cold_start else 0) | (TSID_EXTEND_TC if tensor_cores else 0),
                           stream.cuda_stream, None, 0)
    need = C.c_size_t(0)
    st = lib().tsid_extend_workspace_bytes(C.byref(cfg), col_ptr.data_ptr(), C.byref(need))
    if st != TSID_OK:
        raise TsidError(st, "tsid_extend_workspace_bytes")
    ws = torch.empty(need.value + 256, dtype=torch.uint8, device=dev)
    cfg.workspace = (ws.data_ptr() + 255) & ~255
    cfg.workspace_bytes = need.value
    sse = C.c_double(0)
    with torch.cuda.device(dev):
        st = lib().tsid_extend(C.byref(cfg), P.data_ptr(), Q.data_ptr(), col_ptr.data_ptr(), row_idx.data_ptr(),
                               vals.data_ptr(), C0.data_ptr(), C.byref(sse) if want_sse else None)
    if st != TSID_OK:
        raise TsidError(st, "tsid_extend")
    return sse.value if want_sse else None


def template_from_workload(tpl, path=TSID_PATH_AUTO, flags=0, precision=None) -> Template:
    """Creates a Template from a workloads.Template (device tensors) with its step parameters."""
    w = tpl.w
    prec = precision if precision is not None else (TSID_BF16_SHADOW if w.precision == "bf16" else TSID_F32)
    cfg = make_config(w.m, w.n, w.k, tpl.nnz, prec, path, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q, flags)
    return Template(cfg, tpl.rows, tpl.cols, tpl.vals)
