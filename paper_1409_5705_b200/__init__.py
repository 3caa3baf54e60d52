"""Python binding of libsfb, the B200 (sm_100a) Sufficient Factor Broadcasting step.

Argument marshalling only: every function forwards to the C-ABI entry point of the same name declared in
``include/sfb.h``; all arithmetic runs in the library's CUDA kernels.  PyTorch supplies device memory and
streams.  There is no CPU fallback: loading fails loudly when the library is missing.
"""
from __future__ import annotations

import ctypes
import os

from .build import LIB, build

MLR, DML, SC, L2MLR = 0, 1, 2, 3
PREC_BF16, PREC_FP32, PREC_TF32X3, PREC_FP32_FFMA = 0, 1, 2, 3
PROX_NONE, PROX_L1, PROX_L2SQ = 0, 1, 2
CSR_UPDATE_AUTO, CSR_UPDATE_SPARSE, CSR_UPDATE_DENSE = 0, 1, 2
STATUS_LABEL_RANGE, STATUS_TIMEOUT, STATUS_SAMPLE_RANGE, STATUS_INDEX_RANGE = 0x1, 0x2, 0x4, 0x8

EXPORTS = ("sfb_workspace_bytes", "sfb_init", "sfb_compute_factors", "sfb_gather_factors", "sfb_apply_update",
           "sfb_step", "sfb_step_host", "sfb_dense_sync_step", "sfb_get_factors", "sfb_get_stats",
           "sfb_get_status", "sfb_strerror", "sfb_last_cuda_error", "sfb_destroy", "sfb_prox_columns_noalloc",
           "sfb_selftest_wait_timeout", "sfb_set_row_shard", "sfb_forward_partials", "sfb_finish_factors",
           "sfb_replay_update", "sfb_refresh_operands", "sfb_sdca_set_dual", "sfb_sdca_compute_factors",
           "sfb_sdca_step", "sfb_set_factors", "sfb_set_eta", "sfb_get_operand_copy", "sfb_compute_factors_csr",
           "sfb_step_csr", "sfb_export_factors", "sfb_forward_partials_pairs")
NOALLOC_MAX_COLS = 16384


class sfb_config(ctypes.Structure):
    _fields_ = [("model", ctypes.c_int32), ("precision", ctypes.c_int32), ("rows", ctypes.c_int64),
                ("cols", ctypes.c_int64), ("workers", ctypes.c_int32), ("batch", ctypes.c_int32),
                ("eta", ctypes.c_float), ("dml_margin", ctypes.c_float), ("sc_lambda", ctypes.c_float),
                ("sc_ista_iters", ctypes.c_int32), ("sc_lipschitz", ctypes.c_float), ("sc_prox", ctypes.c_int32),
                ("sdca_lambda", ctypes.c_float), ("sdca_n", ctypes.c_int64), ("prox_kind", ctypes.c_int32),
                ("prox_weight", ctypes.c_float), ("csr_nnz_max", ctypes.c_int64), ("csr_update", ctypes.c_int32), ("stream", ctypes.c_void_p)]


class sfb_stats(ctypes.Structure):
    _fields_ = [("steps", ctypes.c_int64), ("samples", ctypes.c_int64), ("flops", ctypes.c_double),
                ("gather_bytes", ctypes.c_double), ("gather_bytes_p2p", ctypes.c_double),
                ("dense_sync_bytes", ctypes.c_double), ("ms_factors", ctypes.c_float),
                ("ms_gather", ctypes.c_float), ("ms_update", ctypes.c_float), ("last_loss", ctypes.c_float),
                ("sc_lipschitz", ctypes.c_float), ("kernel_launches", ctypes.c_int64),
                ("copy_pieces", ctypes.c_int64), ("copy_written", ctypes.c_int64), ("sparse_updates", ctypes.c_int64)]


class SfbError(RuntimeError):
    def __init__(self, code: int, what: str, cuda: int = 0):
        self.code = code
        self.cuda = cuda
        super().__init__(f"{what}: {strerror(code)} ({code})" + (f", cudaError {cuda}" if cuda else ""))


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB):
            raise RuntimeError(f"{LIB} is missing: run paper_1409_5705_b200.build.build() (needs nvcc); "
                               "there is no fallback path")
        L = ctypes.CDLL(LIB)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        cfgp = ctypes.POINTER(sfb_config)
        L.sfb_workspace_bytes.argtypes = [cfgp, ctypes.POINTER(ctypes.c_size_t)]
        L.sfb_init.argtypes = [cfgp, vp, vp, ctypes.c_size_t, ctypes.POINTER(vp)]
        L.sfb_compute_factors.argtypes = [vp, i32, vp, vp, vp]
        L.sfb_gather_factors.argtypes = [vp]
        L.sfb_apply_update.argtypes = [vp]
        L.sfb_step.argtypes = [vp, vp, vp, vp]
        L.sfb_step_host.argtypes = [vp, vp, vp, vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_uint32)]
        L.sfb_dense_sync_step.argtypes = [vp, vp, vp, vp, vp, ctypes.c_size_t]
        L.sfb_get_factors.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(i32),
                                      ctypes.POINTER(i32), ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.sfb_get_stats.argtypes = [vp, ctypes.POINTER(sfb_stats)]
        L.sfb_get_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
        L.sfb_strerror.argtypes = [ctypes.c_int]
        L.sfb_strerror.restype = ctypes.c_char_p
        L.sfb_last_cuda_error.argtypes = [vp]
        L.sfb_destroy.argtypes = [vp]
        L.sfb_prox_columns_noalloc.argtypes = [vp, i64, i64, vp]
        L.sfb_selftest_wait_timeout.argtypes = [vp, i64]
        L.sfb_set_row_shard.argtypes = [vp, i64, i64]
        L.sfb_forward_partials.argtypes = [vp, vp, vp, vp]
        L.sfb_finish_factors.argtypes = [vp, vp, i32]
        L.sfb_forward_partials_pairs.argtypes = [vp, vp, vp, vp, vp]
        L.sfb_replay_update.argtypes = [vp]
        L.sfb_refresh_operands.argtypes = [vp]
        L.sfb_sdca_set_dual.argtypes = [vp, vp, i64]
        L.sfb_sdca_compute_factors.argtypes = [vp, i32, vp, vp, vp]
        L.sfb_sdca_step.argtypes = [vp, vp, vp, vp]
        L.sfb_set_factors.argtypes = [vp, i32, vp, vp]
        L.sfb_export_factors.argtypes = [vp, i32, vp, vp]
        L.sfb_set_eta.argtypes = [vp, ctypes.c_float]
        L.sfb_get_operand_copy.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(i32), ctypes.POINTER(i64)]
        L.sfb_compute_factors_csr.argtypes = [vp, i32, vp, vp, vp, i64, vp]
        L.sfb_step_csr.argtypes = [vp, vp, vp, vp, i64, vp]
        for name in EXPORTS:
            if name != "sfb_strerror":
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().sfb_strerror(code).decode()


def make_config(model, rows, cols, workers, batch, eta, precision=PREC_FP32, dml_margin=1.0, sc_lambda=0.1,
                sc_ista_iters=20, sc_lipschitz=0.0, sc_prox=0, stream=0, sdca_lambda=0.0, sdca_n=0, prox_kind=0,
                prox_weight=0.0, csr_nnz_max=0, csr_update=0) -> sfb_config:
    return sfb_config(model, precision, rows, cols, workers, batch, eta, dml_margin, sc_lambda, sc_ista_iters,
                      sc_lipschitz, sc_prox, sdca_lambda, sdca_n, prox_kind, prox_weight, csr_nnz_max, csr_update, stream)


def sfb_workspace_bytes(cfg: sfb_config) -> int:
    out = ctypes.c_size_t(0)
    rc = lib().sfb_workspace_bytes(ctypes.byref(cfg), ctypes.byref(out))
    if rc:
        raise SfbError(rc, "sfb_workspace_bytes")
    return out.value


def _ptr(t):
    """Device (or host) address of a torch tensor, an int address, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


class Context:
    """Owns one ``sfb_ctx``.  ``W`` (fp32 CUDA tensor [rows x cols]) is updated in place; the workspace tensor
    is allocated here with torch and kept alive for the life of the context."""

    def __init__(self, cfg: sfb_config, W, stream=None):
        import torch
        assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous()
        assert tuple(W.shape) == (cfg.rows, cfg.cols)
        self.cfg = cfg
        self.W = W
        self.stream = stream if stream is not None else torch.cuda.current_stream(W.device)
        cfg.stream = self.stream.cuda_stream
        nbytes = sfb_workspace_bytes(cfg)
        self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device=W.device)
        base = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        self._h = ctypes.c_void_p()
        rc = lib().sfb_init(ctypes.byref(cfg), W.data_ptr(), base, nbytes, ctypes.byref(self._h))
        if rc:
            raise SfbError(rc, "sfb_init")
        self.K = cfg.workers * cfg.batch

    def _ck(self, rc, what):
        if rc:
            raise SfbError(rc, what, lib().sfb_last_cuda_error(self._h))

    def sfb_compute_factors(self, worker, X, Y=None, labels=None):
        self._ck(lib().sfb_compute_factors(self._h, worker, _ptr(X), _ptr(Y), _ptr(labels)), "sfb_compute_factors")

    def sfb_gather_factors(self):
        self._ck(lib().sfb_gather_factors(self._h), "sfb_gather_factors")

    def sfb_apply_update(self):
        self._ck(lib().sfb_apply_update(self._h), "sfb_apply_update")

    def sfb_sdca_set_dual(self, Q):
        """Q: fp32 CUDA tensor [sdca_n, rows], the dual state (kept alive by the caller; updated in place)."""
        self._dual = Q
        self._ck(lib().sfb_sdca_set_dual(self._h, _ptr(Q), Q.shape[0]), "sfb_sdca_set_dual")

    def sfb_sdca_compute_factors(self, worker, X, labels, sample_ids):
        self._ck(lib().sfb_sdca_compute_factors(self._h, worker, _ptr(X), _ptr(labels), _ptr(sample_ids)),
                 "sfb_sdca_compute_factors")

    def sfb_sdca_step(self, X, labels, sample_ids):
        self._ck(lib().sfb_sdca_step(self._h, _ptr(X), _ptr(labels), _ptr(sample_ids)), "sfb_sdca_step")

    def sfb_set_factors(self, worker, U, V):
        """U [B, rows], V [B, cols]: contiguous fp32 CUDA tensors of factors computed elsewhere."""
        self._ck(lib().sfb_set_factors(self._h, worker, _ptr(U), _ptr(V)), "sfb_set_factors")

    def sfb_export_factors(self, worker, U_out, V_out):
        """U_out [B, rows], V_out [B, cols]: contiguous fp32 CUDA tensors that receive the worker's factors as they are sent."""
        self._ck(lib().sfb_export_factors(self._h, worker, _ptr(U_out), _ptr(V_out)), "sfb_export_factors")

    def sfb_set_eta(self, eta):
        self._ck(lib().sfb_set_eta(self._h, eta), "sfb_set_eta")
        self.cfg.eta = eta

    def sfb_refresh_operands(self):
        self._ck(lib().sfb_refresh_operands(self._h), "sfb_refresh_operands")

    def sfb_replay_update(self):
        self._ck(lib().sfb_replay_update(self._h), "sfb_replay_update")

    def sfb_step(self, X, Y=None, labels=None):
        self._ck(lib().sfb_step(self._h, _ptr(X), _ptr(Y), _ptr(labels)), "sfb_step")

    def sfb_compute_factors_csr(self, worker, indptr, indices, values, nnz, labels):
        """indptr int64 [B+1 or K+1], indices int32, values fp32, labels int32: CUDA tensors; nnz = entries of the call."""
        self._ck(lib().sfb_compute_factors_csr(self._h, worker, _ptr(indptr), _ptr(indices), _ptr(values), nnz,
                                               _ptr(labels)), "sfb_compute_factors_csr")

    def sfb_step_csr(self, indptr, indices, values, nnz, labels):
        self._ck(lib().sfb_step_csr(self._h, _ptr(indptr), _ptr(indices), _ptr(values), nnz, _ptr(labels)), "sfb_step_csr")

    def sfb_step_host(self, X, Y=None, labels=None):
        """X, Y, labels: host tensors / numpy arrays (pinned recommended).  Returns (mean loss, status word)."""
        loss, st = ctypes.c_float(0), ctypes.c_uint32(0)
        self._ck(lib().sfb_step_host(self._h, _host_ptr(X), _host_ptr(Y), _host_ptr(labels), ctypes.byref(loss),
                                     ctypes.byref(st)), "sfb_step_host")
        return loss.value, st.value

    def sfb_dense_sync_step(self, X, Y, labels, scratch):
        self._ck(lib().sfb_dense_sync_step(self._h, _ptr(X), _ptr(Y), _ptr(labels), scratch.data_ptr(),
                                           scratch.numel() * scratch.element_size()), "sfb_dense_sync_step")

    def sfb_get_factors(self):
        """(U address, V address, dtype 0 fp32 / 1 bf16, layout 0 pair-major / 1 transposed, ldu, ldv)."""
        U, V = ctypes.c_void_p(), ctypes.c_void_p()
        dt, lo = ctypes.c_int32(), ctypes.c_int32()
        ldu, ldv = ctypes.c_int64(), ctypes.c_int64()
        self._ck(lib().sfb_get_factors(self._h, ctypes.byref(U), ctypes.byref(V), ctypes.byref(dt), ctypes.byref(lo),
                                       ctypes.byref(ldu), ctypes.byref(ldv)), "sfb_get_factors")
        return U.value, V.value, dt.value, lo.value, ldu.value, ldv.value

    def factors_as_tensors(self):
        """Gathered U [K x rows] and V [K x cols] as fp32 torch tensors (copies; for inspection and tests)."""
        import torch
        U, V, dt, lo, ldu, ldv = self.sfb_get_factors()
        rows, cols, K = self.cfg.rows, self.cfg.cols, self.K
        ws0 = self.workspace.data_ptr()
        tdt = torch.float32 if dt == 0 else torch.bfloat16
        esz = 4 if dt == 0 else 2

        def view(addr, n0, ld):
            off = addr - ws0
            flat = self.workspace[off:off + n0 * ld * esz].view(tdt)
            return flat.view(n0, ld)
        if lo == 0:
            return view(U, K, ldu)[:, :rows].float(), view(V, K, ldv)[:, :cols].float()
        return view(U, rows, ldu)[:, :K].t().float(), view(V, cols, ldv)[:, :K].t().float()

    def capture(self, calls):
        """Captures the library calls made by ``calls()`` on this context's stream into one CUDA graph and returns it
        (``.replay()`` launches them again on the same buffers).  The context must have been created on a stream of
        its own (not the default stream), and every kind of call in ``calls`` must have run once before, so that
        one-off set-up (kernel attributes) is not part of the capture.  Plumbing only: torch records what the library
        launches."""
        import torch
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=self.stream):
            calls()
        return g

    def operand_copy_as_tensor(self):
        """The library's operand copy of W as a torch view into the workspace: bf16 [rows, ld] (MLR, bf16 mode) or
        fp32 [rows, ld] with the (big | small) tf32 halves side by side (tensor-core fp32 mode)."""
        import torch
        ptr, dt, ld = ctypes.c_void_p(), ctypes.c_int32(), ctypes.c_int64()
        self._ck(lib().sfb_get_operand_copy(self._h, ctypes.byref(ptr), ctypes.byref(dt), ctypes.byref(ld)),
                 "sfb_get_operand_copy")
        tdt, esz = (torch.bfloat16, 2) if dt.value == 1 else (torch.float32, 4)
        off = ptr.value - self.workspace.data_ptr()
        return self.workspace[off:off + self.cfg.rows * ld.value * esz].view(tdt).view(self.cfg.rows, ld.value)

    def sfb_get_stats(self) -> sfb_stats:
        st = sfb_stats()
        self._ck(lib().sfb_get_stats(self._h, ctypes.byref(st)), "sfb_get_stats")
        return st

    def sfb_get_status(self) -> int:
        st = ctypes.c_uint32(0)
        self._ck(lib().sfb_get_status(self._h, ctypes.byref(st)), "sfb_get_status")
        return st.value

    def sfb_set_row_shard(self, row_offset, global_rows):
        self._ck(lib().sfb_set_row_shard(self._h, row_offset, global_rows), "sfb_set_row_shard")

    def sfb_forward_partials(self, X, labels, partials):
        """partials: fp32 CUDA tensor [K, 4] that receives this shard's (max, sum exp, label logit, owner flag)."""
        self._ck(lib().sfb_forward_partials(self._h, _ptr(X), _ptr(labels), _ptr(partials)), "sfb_forward_partials")

    def sfb_forward_partials_pairs(self, X, Y, similar, partials):
        self._ck(lib().sfb_forward_partials_pairs(self._h, _ptr(X), _ptr(Y), _ptr(similar), _ptr(partials)),
                 "sfb_forward_partials_pairs")

    def sfb_finish_factors(self, partials_all, shards):
        """partials_all: fp32 CUDA tensor [shards, K, 4], the partials of every shard in shard order."""
        self._ck(lib().sfb_finish_factors(self._h, _ptr(partials_all), shards), "sfb_finish_factors")

    def sfb_selftest_wait_timeout(self, max_cycles):
        self._ck(lib().sfb_selftest_wait_timeout(self._h, max_cycles), "sfb_selftest_wait_timeout")

    def close(self):
        if self._h:
            lib().sfb_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def sfb_prox_columns_noalloc(W, stream=None):
    """Column prox of sparse coding on a CUDA fp32 tensor ``W`` [rows x cols], in place, through the entry point
    that allocates nothing (no context, no workspace: the scratch is an array built into the library).  Argument
    marshalling only; raises SfbError with code -11 when cols exceeds NOALLOC_MAX_COLS."""
    import torch
    assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous() and W.dim() == 2
    st = stream if stream is not None else torch.cuda.current_stream(W.device)
    with torch.cuda.device(W.device):          # the built-in scratch array is per device: W's device must be current
        rc = lib().sfb_prox_columns_noalloc(W.data_ptr(), W.shape[0], W.shape[1], st.cuda_stream)
    if rc:
        raise SfbError(rc, "sfb_prox_columns_noalloc")


def _host_ptr(a):
    if a is None:
        return None
    if hasattr(a, "data_ptr"):
        assert not a.is_cuda
        return a.data_ptr()
    return a.ctypes.data
