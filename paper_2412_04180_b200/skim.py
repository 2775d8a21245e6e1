"""Thin Python binding of libskim.so (argument marshalling only; every step runs in the CUDA
kernels behind the C ABI declared in ``include/skim.h``).

PyTorch is used for device memory and streams.  There is no CPU fallback: loading fails
loudly when the library has not been built, and every call needs CUDA tensors.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# SKIM_LIB selects another build of the same library (the bounds-checked one, build.py --checked)
LIB_PATH = os.environ.get("SKIM_LIB") or os.path.join(_HERE, "libskim.so")
_lib = None

ERR_NAMES = {0: "SKIM_OK", -1: "SKIM_ERR_NULL", -2: "SKIM_ERR_SHAPE", -3: "SKIM_ERR_BITSET",
             -4: "SKIM_ERR_BUDGET", -5: "SKIM_ERR_WORKSPACE", -6: "SKIM_ERR_CUDA",
             -7: "SKIM_ERR_BAD_DATA", -8: "SKIM_ERR_SCALE", -9: "SKIM_ERR_ALIGN", -10: "SKIM_ERR_STATIC_LIMIT"}

EXPORTS = ["skim_create", "skim_destroy", "skim_max_cols", "skim_workspace_bytes", "skim_set_workspace",
           "skim_apply_scale", "skim_cluster_rows", "skim_cluster_rows_at", "skim_cluster_exact_bytes", "skim_cluster_rows_exact", "skim_allocate_bits", "skim_allocate_bits_floor", "skim_allocate_bits_until", "skim_allocate_optimal_bytes", "skim_allocate_optimal",
           "skim_packed_layout", "skim_quantize", "skim_quantize_static", "skim_dequantize", "skim_matvec", "skim_scale_update", "skim_scale_lfull_bytes", "skim_scale_update_lfull", "skim_residual", "skim_err_lfull_bytes", "skim_err_lfull", "skim_host_staging_bytes",
           "skim_quantize_matrix_host", "skim_get_status", "skim_launch_count", "skim_kernel_timing",
           "skim_kernel_times", "skim_early_exit", "skim_lloyd_iterations", "skim_strerror"]


class SkimError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        msg = lib().skim_strerror(code).decode()
        super().__init__(f"{where}: {ERR_NAMES.get(code, code)} ({msg})")


def lib():
    """Loads libskim.so; raises if it is missing (build it with ``python -m paper_2412_04180_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: the CUDA library has not been built "
                               "(run `python -m paper_2412_04180_b200.build`); there is no fallback")
        _lib = C.CDLL(LIB_PATH)
        _lib.skim_strerror.restype = C.c_char_p
        _lib.skim_strerror.argtypes = [C.c_int]
        _lib.skim_launch_count.restype = C.c_int64
        _lib.skim_launch_count.argtypes = [C.c_void_p]
    return _lib


def _ptr(t):
    if t is None:
        return C.c_void_p(0)
    return C.c_void_p(t.data_ptr())


def _bits(bit_set):
    arr = (C.c_int * len(bit_set))(*[int(b) for b in bit_set])
    return arr, len(bit_set), sum(1 << int(b) for b in bit_set)


def _chk(rc, where):
    if rc != 0:
        raise SkimError(rc, where)


def _dev(t, dtype, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of dtype {dtype}")
    return t


class Skim:
    """One context: a device, a stream and a caller-owned workspace."""

    def __init__(self, device=0, stream=None, rows=0, cols=0):
        self.device = torch.device("cuda", device)
        self._stream = stream
        handle = C.c_void_p()
        sp = C.c_void_p(stream.cuda_stream if stream is not None else 0)
        _chk(lib().skim_create(C.byref(handle), C.c_int(device), sp), "skim_create")
        self._h = handle
        self._ws = None
        self._scale = None      # the installed scale vector (kept so that a new workspace can take it over)
        if rows and cols:
            self.reserve(rows, cols)

    def close(self):
        if self._h is not None:
            lib().skim_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- workspace
    def max_cols(self):
        out = C.c_int64()
        _chk(lib().skim_max_cols(self._h, C.byref(out)), "skim_max_cols")
        return out.value

    @staticmethod
    def workspace_bytes(rows, cols):
        out = C.c_size_t()
        _chk(lib().skim_workspace_bytes(C.c_int64(rows), C.c_int64(cols), C.byref(out)), "skim_workspace_bytes")
        return out.value

    def reserve(self, rows, cols):
        """Allocates (with torch) and installs a workspace big enough for rows x cols.  A scale vector
        that is installed moves to the new workspace with it."""
        nbytes = self.workspace_bytes(rows, cols)
        if self._ws is None or self._ws.numel() < nbytes:
            if self._ws is not None:
                # work already enqueued on the context's stream may still use the old buffer
                (self._stream.synchronize() if self._stream is not None else torch.cuda.synchronize(self.device))
            self.set_workspace(torch.empty(nbytes, dtype=torch.uint8, device=self.device))

    def set_workspace(self, buf):
        """Installs a caller-owned workspace.  skim_set_workspace drops an installed scale vector (its
        reciprocal lives in the old workspace), so the binding installs it again in the new one."""
        _dev(buf, torch.uint8, "workspace")
        _chk(lib().skim_set_workspace(self._h, _ptr(buf), C.c_size_t(buf.numel())), "skim_set_workspace")
        self._ws = buf
        if self._scale is not None:
            self.apply_scale(self._scale)

    # ---- the path
    def apply_scale(self, s, cols=None):
        if s is None:
            _chk(lib().skim_apply_scale(self._h, C.c_void_p(0), C.c_int64(0)), "skim_apply_scale")
            self._scale = None
            return
        _dev(s, torch.float32, "s")
        _chk(lib().skim_apply_scale(self._h, _ptr(s), C.c_int64(s.numel() if cols is None else cols)),
             "skim_apply_scale")
        self._scale = s.clone() if cols is None else None     # a copy: callers update their vector in place

    def cluster_rows(self, W, importance, bit_set, iters, want_centroids=True, want_codes=False, ld=None,
                     cols=None):
        """Returns (centroids [rows, sumk] or None, codes [n_bits, rows, cols] or None, err [rows, n_bits])."""
        _dev(W, torch.float16, "W")
        _dev(importance, torch.float32, "importance")
        rows = W.shape[0]
        ld = W.shape[1] if ld is None else ld
        cols = W.shape[1] if cols is None else cols
        arr, nb, sumk = _bits(bit_set)
        cent = torch.empty((rows, sumk), dtype=torch.float32, device=W.device) if want_centroids else None
        codes = torch.empty((nb, rows, cols), dtype=torch.uint8, device=W.device) if want_codes else None
        err = torch.empty((rows, nb), dtype=torch.float32, device=W.device)
        _chk(lib().skim_cluster_rows(self._h, _ptr(W), _ptr(importance), C.c_int64(rows), C.c_int64(cols),
                                     C.c_int64(ld), arr, C.c_int(nb), C.c_int(iters), _ptr(cent), _ptr(codes),
                                     _ptr(err)), "skim_cluster_rows")
        return cent, codes, err

    def cluster_rows_into(self, W, importance, bit_set, iters, centroids, err, codes=None):
        """As cluster_rows, writing into caller-provided tensors (no allocation; used when timing)."""
        rows, cols = W.shape
        arr, nb, _ = _bits(bit_set)
        _chk(lib().skim_cluster_rows(self._h, _ptr(W), _ptr(importance), C.c_int64(rows), C.c_int64(cols),
                                     C.c_int64(cols), arr, C.c_int(nb), C.c_int(iters), _ptr(centroids),
                                     _ptr(codes), _ptr(err)), "skim_cluster_rows")

    def cluster_rows_at(self, W, importance, row_bits, bit_set, iters, want_codes=True, centroids=None):
        """Returns (centroids [rows, sumk], codes [rows, cols] or None, err [rows])."""
        _dev(W, torch.float16, "W")
        _dev(importance, torch.float32, "importance")
        _dev(row_bits, torch.uint8, "row_bits")
        rows, cols = W.shape
        arr, nb, sumk = _bits(bit_set)
        cent = centroids if centroids is not None else torch.zeros((rows, sumk), dtype=torch.float32, device=W.device)
        codes = torch.empty((rows, cols), dtype=torch.uint8, device=W.device) if want_codes else None
        err = torch.empty((rows,), dtype=torch.float32, device=W.device)
        _chk(lib().skim_cluster_rows_at(self._h, _ptr(W), _ptr(importance), C.c_int64(rows), C.c_int64(cols),
                                        C.c_int64(cols), _ptr(row_bits), arr, C.c_int(nb), C.c_int(iters),
                                        _ptr(cent), _ptr(codes), _ptr(err)), "skim_cluster_rows_at")
        return cent, codes, err

    def cluster_rows_exact(self, W, importance, bit_set, scratch=None):
        """The optimum of the clustering objective per row: returns (centroids [rows, sumk], err [rows, n_bits])."""
        _dev(W, torch.float16, "W")
        _dev(importance, torch.float32, "importance")
        rows, cols = W.shape
        arr, nb, sumk = _bits(bit_set)
        need = C.c_size_t()
        _chk(lib().skim_cluster_exact_bytes(self._h, C.c_int64(rows), C.c_int64(cols), C.byref(need)), "skim_cluster_exact_bytes")
        if scratch is None:
            scratch = torch.empty(need.value, dtype=torch.uint8, device=W.device)
        cent = torch.empty((rows, sumk), dtype=torch.float32, device=W.device)
        err = torch.empty((rows, nb), dtype=torch.float32, device=W.device)
        _chk(lib().skim_cluster_rows_exact(self._h, _ptr(W), _ptr(importance), C.c_int64(rows), C.c_int64(cols),
                                           C.c_int64(cols), arr, C.c_int(nb), _ptr(scratch), C.c_size_t(scratch.numel()),
                                           _ptr(cent), _ptr(err)), "skim_cluster_rows_exact")
        return cent, err

    def allocate_bits(self, err, bit_set, budget, out=None, floor_start=False, round_up=False):
        """Returns (bits uint8 [rows], total_bits).  floor_start: every row starts at floor(budget)
        instead of the smallest width (skim_allocate_bits_floor).  round_up: the total is rounded up, Algorithm 1's
        stopping rule as printed (skim_allocate_bits_until)."""
        _dev(err, torch.float32, "err")
        rows = err.shape[0]
        arr, nb, _ = _bits(bit_set)
        bits = out if out is not None else torch.empty((rows,), dtype=torch.uint8, device=err.device)
        total = C.c_int64()
        fn = lib().skim_allocate_bits_floor if floor_start else lib().skim_allocate_bits
        if round_up:
            fn = lib().skim_allocate_bits_until
        _chk(fn(self._h, _ptr(err), C.c_int64(rows), arr, C.c_int(nb), C.c_double(budget), _ptr(bits), C.byref(total)),
             "skim_allocate_bits_floor" if floor_start else "skim_allocate_bits")
        return bits, total.value

    def allocate_optimal(self, err, bit_set, budget):
        """Exact minimum-error allocation (dynamic programme); returns (bits uint8 [rows], total_bits, cost)."""
        _dev(err, torch.float32, "err")
        rows = err.shape[0]
        arr, nb, _ = _bits(bit_set)
        need = C.c_size_t()
        _chk(lib().skim_allocate_optimal_bytes(C.c_int64(rows), arr, C.c_int(nb), C.c_double(budget), C.byref(need)),
             "skim_allocate_optimal_bytes")
        scratch = torch.empty(need.value, dtype=torch.uint8, device=err.device)
        bits = torch.empty((rows,), dtype=torch.uint8, device=err.device)
        cost = torch.zeros((1,), dtype=torch.float64, device=err.device)
        total = C.c_int64()
        _chk(lib().skim_allocate_optimal(self._h, _ptr(err), C.c_int64(rows), arr, C.c_int(nb), C.c_double(budget),
                                         _ptr(scratch), C.c_size_t(need.value), _ptr(bits), C.byref(total), _ptr(cost)),
             "skim_allocate_optimal")
        return bits, total.value, float(cost.item())

    @staticmethod
    def packed_layout(rows, cols, bit_set):
        """Returns (row stride in 32-bit words for every width, max packed bytes)."""
        arr, nb, _ = _bits(bit_set)
        strides = (C.c_int64 * nb)()
        mx = C.c_size_t()
        _chk(lib().skim_packed_layout(C.c_int64(rows), C.c_int64(cols), arr, C.c_int(nb), strides, C.byref(mx)),
             "skim_packed_layout")
        return list(strides), mx.value

    def quantize(self, W, bits, centroids, bit_set, out=None):
        """Returns dict(packed uint32 (max size), row_order int32 [rows], group_info int64 [2*(n_bits+1)],
        lut uint16 [rows, 2^b_max])."""
        _dev(W, torch.float16, "W")
        _dev(bits, torch.uint8, "bits")
        _dev(centroids, torch.float32, "centroids")
        rows, cols = W.shape
        arr, nb, _ = _bits(bit_set)
        if out is None:
            _, mx = self.packed_layout(rows, cols, bit_set)
            out = dict(packed=torch.empty(mx // 4, dtype=torch.int32, device=W.device),
                       row_order=torch.empty(rows, dtype=torch.int32, device=W.device),
                       group_info=torch.empty(2 * (nb + 1), dtype=torch.int64, device=W.device),
                       lut=torch.empty((rows, 1 << int(bit_set[-1])), dtype=torch.int16, device=W.device))
        _chk(lib().skim_quantize(self._h, _ptr(W), C.c_int64(rows), C.c_int64(cols), C.c_int64(cols), _ptr(bits),
                                 _ptr(centroids), arr, C.c_int(nb), _ptr(out["packed"]), _ptr(out["row_order"]),
                                 _ptr(out["group_info"]), _ptr(out["lut"])), "skim_quantize")
        return out

    def dequantize(self, q, cols, bit_set, s=None, out=None):
        """float16 [rows, cols] dequantised weights from a quantize() result ``q``; ``s`` is the scaling vector."""
        rows = q["row_order"].numel()
        arr, nb, _ = _bits(bit_set)
        if s is not None:
            _dev(s, torch.float32, "s")
        if out is None:
            out = torch.empty((rows, cols), dtype=torch.float16, device=q["packed"].device)
        _chk(lib().skim_dequantize(self._h, _ptr(q["packed"]), _ptr(q["row_order"]), _ptr(q["group_info"]),
                                   _ptr(q["lut"]), _ptr(s), C.c_int64(rows), C.c_int64(cols), arr, C.c_int(nb),
                                   _ptr(out), C.c_int64(out.stride(0))), "skim_dequantize")
        return out

    def matvec(self, q, cols, bit_set, x, s=None, out=None):
        """float32 [rows] = Wq x from a quantize() result ``q`` and a float16 vector ``x`` [cols]."""
        rows = q["row_order"].numel()
        arr, nb, _ = _bits(bit_set)
        _dev(x, torch.float16, "x")
        if s is not None:
            _dev(s, torch.float32, "s")
        if out is None:
            out = torch.empty((rows,), dtype=torch.float32, device=x.device)
        _chk(lib().skim_matvec(self._h, _ptr(q["packed"]), _ptr(q["row_order"]), _ptr(q["group_info"]), _ptr(q["lut"]),
                               _ptr(s), _ptr(x), C.c_int64(rows), C.c_int64(cols), arr, C.c_int(nb), _ptr(out)),
             "skim_matvec")
        return out

    def scale_update(self, W, importance, labels, alpha, steps=120, lr0=0.01, decay=0.5, decay_every=40,
                     want_trace=True):
        """Updates alpha (float32 CUDA tensor) in place; returns the loss trace (float64 [steps]) or None."""
        _dev(W, torch.float16, "W")
        _dev(importance, torch.float32, "importance")
        _dev(labels, torch.uint8, "labels")
        _dev(alpha, torch.float32, "alpha")
        rows, cols = W.shape
        trace = torch.zeros(max(steps, 1), dtype=torch.float64, device=W.device) if want_trace else None
        _chk(lib().skim_scale_update(self._h, _ptr(W), _ptr(importance), C.c_int64(rows), C.c_int64(cols),
                                     C.c_int64(cols), _ptr(labels), _ptr(alpha), C.c_int(steps), C.c_float(lr0),
                                     C.c_float(decay), C.c_int(decay_every), _ptr(trace)), "skim_scale_update")
        return trace[:steps] if want_trace else None

    def scale_update_lfull(self, W, importance, labels, alpha, H, steps=120, lr0=0.01, decay=0.5, decay_every=40, exp2=8,
                           want_trace=True, scratch=None):
        """scale_update on the L-full loss with Gram matrix H (float16 [cols, cols]); alpha is updated in place."""
        _dev(W, torch.float16, "W")
        _dev(importance, torch.float32, "importance")
        _dev(labels, torch.uint8, "labels")
        _dev(alpha, torch.float32, "alpha")
        _dev(H, torch.float16, "H")
        rows, cols = W.shape
        need = C.c_size_t()
        _chk(lib().skim_scale_lfull_bytes(C.c_int64(rows), C.c_int64(cols), C.byref(need)), "skim_scale_lfull_bytes")
        if scratch is None:
            scratch = torch.empty(need.value, dtype=torch.uint8, device=W.device)
        trace = torch.zeros(max(steps, 1), dtype=torch.float64, device=W.device) if want_trace else None
        _chk(lib().skim_scale_update_lfull(self._h, _ptr(W), _ptr(importance), C.c_int64(rows), C.c_int64(cols),
                                           C.c_int64(cols), _ptr(labels), _ptr(H), C.c_int64(H.stride(0)), _ptr(alpha),
                                           C.c_int(steps), C.c_float(lr0), C.c_float(decay), C.c_int(decay_every),
                                           C.c_int(exp2), _ptr(scratch), C.c_size_t(scratch.numel()), _ptr(trace)),
             "skim_scale_update_lfull")
        return trace[:steps] if want_trace else None

    def residual(self, W, centroids, bit_set, width=None, row_bits=None, s=None, exp2=8, out=None):
        """float16 [rows, cols] scaled residual (W - c[label] * alpha) * 2^exp2, the operand of err_lfull."""
        _dev(W, torch.float16, "W")
        _dev(centroids, torch.float32, "centroids")
        rows, cols = W.shape
        arr, nb, _ = _bits(bit_set)
        if row_bits is not None:
            _dev(row_bits, torch.uint8, "row_bits")
        if s is not None:
            _dev(s, torch.float32, "s")
        if out is None:
            out = torch.empty((rows, cols), dtype=torch.float16, device=W.device)
        _chk(lib().skim_residual(self._h, _ptr(W), C.c_int64(rows), C.c_int64(cols), C.c_int64(cols), _ptr(centroids),
                                 _ptr(row_bits), C.c_int(0 if width is None else int(width)), arr, C.c_int(nb), _ptr(s),
                                 C.c_int(exp2), _ptr(out), C.c_int64(out.stride(0))), "skim_residual")
        return out

    @staticmethod
    def err_lfull_bytes(rows, cols):
        out = C.c_size_t()
        _chk(lib().skim_err_lfull_bytes(C.c_int64(rows), C.c_int64(cols), C.byref(out)), "skim_err_lfull_bytes")
        return out.value

    def err_lfull(self, D, H, exp2=8, scratch=None, out=None, out_stride=1):
        """float32 [rows] L-full errors d H d^T / 4^exp2 of the rows of D (float16) for H (float16 [cols, cols])."""
        _dev(D, torch.float16, "D")
        _dev(H, torch.float16, "H")
        rows, cols = D.shape
        need = self.err_lfull_bytes(rows, cols)
        if scratch is None:
            scratch = torch.empty(need, dtype=torch.uint8, device=D.device)
        if out is None:
            out = torch.empty((rows,), dtype=torch.float32, device=D.device)
        _chk(lib().skim_err_lfull(self._h, _ptr(D), C.c_int64(rows), C.c_int64(cols), C.c_int64(D.stride(0)), _ptr(H),
                                  C.c_int64(H.stride(0)), C.c_int(exp2), _ptr(scratch), C.c_size_t(scratch.numel()),
                                  _ptr(out), C.c_int64(out_stride)), "skim_err_lfull")
        return out

    @staticmethod
    def host_staging_bytes(rows, cols, bit_set):
        arr, nb, _ = _bits(bit_set)
        out = C.c_size_t()
        _chk(lib().skim_host_staging_bytes(C.c_int64(rows), C.c_int64(cols), arr, C.c_int(nb), C.byref(out)),
             "skim_host_staging_bytes")
        return out.value

    def quantize_matrix_host(self, W_host, importance_host, bit_set, iters, budget, staging, out):
        """Whole path from pinned host tensors; ``out`` holds pinned host tensors err, bits, packed,
        row_order, group_info, lut (any may be missing)."""
        rows, cols = W_host.shape
        arr, nb, _ = _bits(bit_set)
        g = lambda k: _ptr(out.get(k))
        _chk(lib().skim_quantize_matrix_host(self._h, _ptr(W_host), _ptr(importance_host), C.c_int64(rows),
                                             C.c_int64(cols), arr, C.c_int(nb), C.c_int(iters), C.c_double(budget),
                                             _ptr(staging), C.c_size_t(staging.numel()), g("err"), g("bits"),
                                             g("packed"), g("row_order"), g("group_info"), g("lut")),
             "skim_quantize_matrix_host")

    def get_status(self):
        """Returns the status flags (and clears them); 0 means no bad data was seen."""
        flags = C.c_uint64()
        rc = lib().skim_get_status(self._h, C.byref(flags))
        if rc not in (0, -7):
            raise SkimError(rc, "skim_get_status")
        return flags.value

    def launch_count(self):
        return int(lib().skim_launch_count(self._h))

    def kernel_timing(self, enable=True):
        """Starts (or stops) recording CUDA events around the sort and Lloyd kernels of every clustering chunk."""
        _chk(lib().skim_kernel_timing(self._h, C.c_int(1 if enable else 0)), "skim_kernel_timing")

    def kernel_times(self):
        """Returns (sort kernel ms, Lloyd kernel ms, chunks) summed since kernel_timing(True); waits for the events."""
        s, l, n = C.c_double(), C.c_double(), C.c_int64()
        _chk(lib().skim_kernel_times(self._h, C.byref(s), C.byref(l), C.byref(n)), "skim_kernel_times")
        return s.value, l.value, n.value


    def early_exit(self, enable=True):
        """Measurement aid: rows stop iterating once no boundary moved (default) or always run all iterations."""
        _chk(lib().skim_early_exit(self._h, C.c_int(1 if enable else 0)), "skim_early_exit")

    def lloyd_iterations(self):
        """Returns (iterations summed over rows, rows counted) since the last call, while kernel_timing is on."""
        it, n = C.c_int64(), C.c_int64()
        _chk(lib().skim_lloyd_iterations(self._h, C.byref(it), C.byref(n)), "skim_lloyd_iterations")
        return it.value, n.value


STATIC_MAX_ROWS = 65536


def quantize_static(W, bits, centroids, bit_set, out, stream=None):
    """skim_quantize_static: the packer for callers that must not allocate device memory.

    No context and no workspace are involved; the scratch is a fixed array inside the library.
    ``out`` must hold preallocated CUDA tensors ``packed``, ``row_order``, ``group_info`` and
    ``lut`` (this wrapper allocates nothing either).  Runs on the current device and on
    ``stream`` (default: torch's current stream).  Calls that overlap on the GPU race on the
    shared scratch, so keep them on one stream.
    """
    _dev(W, torch.float16, "W")
    _dev(bits, torch.uint8, "bits")
    _dev(centroids, torch.float32, "centroids")
    rows, cols = W.shape
    arr, nb, _ = _bits(bit_set)
    st = stream if stream is not None else torch.cuda.current_stream()
    _chk(lib().skim_quantize_static(C.c_void_p(st.cuda_stream), _ptr(W), C.c_int64(rows), C.c_int64(cols),
                                    C.c_int64(cols), _ptr(bits), _ptr(centroids), arr, C.c_int(nb),
                                    _ptr(out["packed"]), _ptr(out["row_order"]), _ptr(out["group_info"]),
                                    _ptr(out["lut"])), "skim_quantize_static")
    return out
