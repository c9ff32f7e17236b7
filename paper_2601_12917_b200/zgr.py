"""ctypes binding of the ZGR C ABI (``include/zgr.h``).

Argument marshalling only: every step of the path (generator, Gaussian transform, ``U G``
synthesis, the in-place sweeps, the norm bookkeeping) runs in the CUDA library.  torch tensors
are used for device memory and streams; the library sees raw pointers.  If ``libzgr.so`` is
missing the import of the library fails loudly -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("ZGR_LIBRARY", os.path.join(_HERE, "libzgr.so"))   # override: an alternative build of the same ABI

OK, EINVAL, ESTATE, ECUDA, ENOMEM, ETOOBIG = 0, -1, -2, -3, -4, -5
NOALLOC_MAX_TILES = 8192
F32, F16, BF16 = 0, 1, 2
SCALE_PAPER, SCALE_UNIT = 0, 1
TAG_ISO, TAG_COEFF = 0, 1
MAX_RANK = 64


class ZgrTensor(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64), ("dtype", ctypes.c_int32),
                ("rank", ctypes.c_int32), ("U", ctypes.c_void_p)]


class ZgrConfig(ctypes.Structure):
    _fields_ = [("alpha", ctypes.c_double), ("eps", ctypes.c_double), ("scale_mode", ctypes.c_int32), ("bits_per_normal", ctypes.c_int32),
                ("stats", ctypes.c_int32)]


class ZgrCoeffDelivery(ctypes.Structure):
    _fields_ = [("tensor", ctypes.c_int32), ("q", ctypes.c_void_p), ("scale", ctypes.c_void_p), ("zero", ctypes.c_void_p), ("U", ctypes.c_void_p)]


class ZgrKernelTime(ctypes.Structure):
    _fields_ = [("path", ctypes.c_int32), ("dtype", ctypes.c_int32), ("kpad", ctypes.c_int32), ("launches", ctypes.c_int32),
                ("elements", ctypes.c_int64), ("ms_total", ctypes.c_double)]


PATH_NAMES = {0: "iso", 1: "fma", 2: "mma", 3: "generic", 4: "umma"}


class ZgrError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


_lib = None


def lib() -> ctypes.CDLL:
    """Load ``libzgr.so`` (built in-tree by ``paper_2601_12917_b200/build.py``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2601_12917_b200.build` "
                              "(there is no CPU fallback for the ZGR step)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, u64, dbl = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_double
        L.zgr_init.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(ZgrTensor), i32, ctypes.POINTER(ZgrConfig)]
        L.zgr_perturb.argtypes = [vp, u64, dbl, vp]
        L.zgr_restore_update.argtypes = [vp, u64, dbl, dbl, dbl, vp]
        L.zgr_sweep_multi.argtypes = [vp, i32, ctypes.POINTER(u64), ctypes.POINTER(dbl), vp]
        L.zgr_restore_update_multi.argtypes = [vp, i32, ctypes.POINTER(u64), ctypes.POINTER(dbl), ctypes.POINTER(dbl), dbl, vp]
        L.zgr_set_coeffs_dtc.argtypes = [vp, i32, vp, vp, vp, i32]
        L.zgr_set_alpha.argtypes = [vp, dbl]
        L.zgr_clear_coeffs.argtypes = [vp, i32]
        L.zgr_get_stats.argtypes = [vp, u64, ctypes.POINTER(dbl), vp]
        L.zgr_debug_philox.argtypes = [vp, u64, i32, i32, u64, i64, vp, vp]
        L.zgr_debug_z.argtypes = [vp, u64, i32, vp, vp]
        L.zgr_debug_z_tcgen05.argtypes = [vp, u64, i32, vp, vp]
        L.zgr_debug_z_tcgen05.restype = ctypes.c_int
        L.zgr_debug_check_device.argtypes = [i32, i32]
        L.zgr_debug_check_device.restype = ctypes.c_int
        L.zgr_adapt_alpha.argtypes = [vp, ctypes.POINTER(dbl), dbl, dbl, dbl, ctypes.POINTER(dbl)]
        L.zgr_adapt_alpha.restype = ctypes.c_int
        L.zgr_build_subspace.argtypes = [vp, i32, vp, i32, vp]
        L.zgr_build_subspace.restype = ctypes.c_int
        L.zgr_enable_stats.argtypes = [vp, i32]
        L.zgr_enable_stats.restype = ctypes.c_int
        L.zgr_set_coeffs_dtc_rows.argtypes = [vp, i32, vp, vp, vp, i32, i32]
        L.zgr_set_coeffs_dtc_rows.restype = ctypes.c_int
        L.zgr_perturb_layers.argtypes = [vp, u64, dbl, i32, ctypes.POINTER(i32), i32, ctypes.POINTER(ZgrCoeffDelivery), vp, vp]
        L.zgr_perturb_layers.restype = ctypes.c_int
        L.zgr_get_scalars.argtypes = [vp, ctypes.POINTER(dbl), ctypes.POINTER(dbl)]
        L.zgr_get_state.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(u64), ctypes.POINTER(dbl)]
        L.zgr_update_subspace.argtypes = [vp, i32, vp, i32, vp]
        L.zgr_update_subspaces.argtypes = [vp, i32, ctypes.POINTER(i32), ctypes.POINTER(vp), i32, vp]
        L.zgr_update_subspaces.restype = ctypes.c_int
        L.zgr_profile.argtypes = [vp, i32]
        L.zgr_profile_read.argtypes = [vp, ctypes.POINTER(ZgrKernelTime), i32, ctypes.POINTER(i32)]
        L.zgr_tensor_norms_noalloc.argtypes = [vp, u64, i32, vp, vp]
        L.zgr_tensor_norms_noalloc.restype = ctypes.c_int
        L.zgr_device_status.argtypes = [vp, ctypes.POINTER(i32)]
        L.zgr_device_status.restype = ctypes.c_int
        L.zgr_launch_count.argtypes = [vp]
        L.zgr_launch_count.restype = i64
        L.zgr_destroy.argtypes = [vp]
        L.zgr_destroy.restype = None
        L.zgr_strerror.argtypes = [ctypes.c_int]
        L.zgr_strerror.restype = ctypes.c_char_p
        for name in ("zgr_init", "zgr_perturb", "zgr_restore_update", "zgr_set_coeffs_dtc", "zgr_clear_coeffs", "zgr_get_stats",
                     "zgr_debug_philox", "zgr_debug_z", "zgr_get_scalars", "zgr_get_state", "zgr_update_subspace", "zgr_profile",
                     "zgr_profile_read", "zgr_sweep_multi", "zgr_restore_update_multi", "zgr_set_alpha"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().zgr_strerror(code).decode()


def _check(code: int, what: str) -> None:
    if code != OK:
        raise ZgrError(code, what)


def _dtype_code(t) -> int:
    import torch
    return {torch.float32: F32, torch.float16: F16, torch.bfloat16: BF16}[t.dtype]


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


class Zgr:
    """A ZGR context over a list of device tensors (``zgr_init`` ... ``zgr_destroy``).

    ``weights[l]`` is a contiguous CUDA tensor (1-D or 2-D; fp32, fp16 or bf16) updated in place;
    ``subspaces[l]`` is ``None`` or a contiguous fp32 CUDA tensor of shape (rows, rank) with
    orthonormal columns.  The context keeps references to all of them.
    """

    def __init__(self, weights: Sequence, subspaces: Sequence, alpha: float, eps: float, scale_mode: int = SCALE_UNIT,
                 bits_per_normal: int = 32, stats: bool = False):
        assert len(weights) == len(subspaces)
        self._keep: List = [list(weights), list(subspaces)]
        n = len(weights)
        arr = (ZgrTensor * n)()
        for l, (w, U) in enumerate(zip(weights, subspaces)):
            if not w.is_cuda or not w.is_contiguous():
                raise ValueError(f"tensor {l}: weights must be contiguous CUDA tensors")
            rows, cols = (1, w.numel()) if w.dim() == 1 else (w.shape[0], w.shape[1])
            rank = 0
            uptr = None
            if U is not None:
                if not U.is_cuda or not U.is_contiguous() or U.shape[0] != rows:
                    raise ValueError(f"tensor {l}: subspace must be a contiguous CUDA tensor of shape (rows, rank)")
                rank, uptr = int(U.shape[1]), U.data_ptr()
            arr[l] = ZgrTensor(w.data_ptr(), rows, cols, _dtype_code(w), rank, uptr)
        cfg = ZgrConfig(alpha, eps, scale_mode, bits_per_normal, 1 if stats else 0)
        self._h = ctypes.c_void_p()
        _check(lib().zgr_init(ctypes.byref(self._h), arr, n, ctypes.byref(cfg)), "zgr_init")
        self.n = n

    # -- the three calls of a step --------------------------------------------------------------
    def perturb(self, seed: int, scale: float, stream=None) -> None:
        _check(lib().zgr_perturb(self._h, seed, scale, _stream_ptr(stream)), "zgr_perturb")

    def restore_update(self, seed: int, loss_plus: float, loss_minus: float, lr: float, stream=None) -> None:
        _check(lib().zgr_restore_update(self._h, seed, loss_plus, loss_minus, lr, _stream_ptr(stream)), "zgr_restore_update")

    # -- several seeds in one sweep ---------------------------------------------------------------
    def sweep_multi(self, seeds: Sequence[int], coeffs: Sequence[float], stream=None) -> None:
        """theta <- rnd(theta + sum_i coeffs[i] z(seeds[i])) in one pass (zgr_sweep_multi)."""
        n = len(seeds)
        assert n == len(coeffs)
        _check(lib().zgr_sweep_multi(self._h, n, (ctypes.c_uint64 * n)(*seeds), (ctypes.c_double * n)(*coeffs), _stream_ptr(stream)),
               "zgr_sweep_multi")

    def restore_update_multi(self, seeds: Sequence[int], loss_plus: Sequence[float], loss_minus: Sequence[float], lr: float, stream=None) -> None:
        """Restore and projected-gradient update of several seeds in one pass (zgr_restore_update_multi)."""
        n = len(seeds)
        assert n == len(loss_plus) == len(loss_minus)
        _check(lib().zgr_restore_update_multi(self._h, n, (ctypes.c_uint64 * n)(*seeds), (ctypes.c_double * n)(*loss_plus),
                                              (ctypes.c_double * n)(*loss_minus), lr, _stream_ptr(stream)), "zgr_restore_update_multi")

    def set_alpha(self, alpha: float) -> None:
        """New mixing ratio for the following steps (zgr_set_alpha)."""
        _check(lib().zgr_set_alpha(self._h, alpha), "zgr_set_alpha")

    def adapt_alpha(self, stats, alpha_min: float = 0.05, alpha_max: float = 0.95, eta: float = 1.0) -> float:
        """Move the mixing ratio towards the balance of the two parts' energies (zgr_adapt_alpha); `stats` is
        the array returned by get_stats under the current ratio.  Returns the new ratio."""
        import numpy as np
        st = np.ascontiguousarray(stats, dtype=np.float64).reshape(-1)
        assert st.size == 3 * self.n
        out = ctypes.c_double()
        _check(lib().zgr_adapt_alpha(self._h, st.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), alpha_min, alpha_max, eta, ctypes.byref(out)),
               "zgr_adapt_alpha")
        return out.value

    def build_subspace(self, tensor: int, grads=None, stream=None) -> None:
        """Orthonormal basis of the span of the gradient directions `grads` (rows x rank fp32 torch tensor on the
        host or on the device; None if they were written into the subspace buffer) becomes the subspace of
        `tensor` (zgr_build_subspace)."""
        if grads is None:
            ptr, host = None, 0
        else:
            assert grads.is_contiguous() and grads.dtype == self._keep[1][tensor].dtype and grads.shape == self._keep[1][tensor].shape
            ptr, host = grads.data_ptr(), 0 if grads.is_cuda else 1
        _check(lib().zgr_build_subspace(self._h, tensor, ptr, host, _stream_ptr(stream)), "zgr_build_subspace")

    # -- compressed coefficients ----------------------------------------------------------------
    def set_coeffs_dtc(self, tensor: int, q, scale, zero=None, bits: int = 8) -> None:
        self._keep.append((q, scale, zero))
        _check(lib().zgr_set_coeffs_dtc(self._h, tensor, q.data_ptr(), scale.data_ptr(), None if zero is None else zero.data_ptr(), bits),
               "zgr_set_coeffs_dtc")

    def set_coeffs_dtc_rows(self, tensor: int, q, scale, zero, bits: int, n_rows: int) -> None:
        """Only the first n_rows rows of the tensor's coefficients come from codes (zgr_set_coeffs_dtc_rows)."""
        self._keep.append((q, scale, zero))
        _check(lib().zgr_set_coeffs_dtc_rows(self._h, tensor, q.data_ptr(), scale.data_ptr(), None if zero is None else zero.data_ptr(), bits, n_rows),
               "zgr_set_coeffs_dtc_rows")

    def perturb_layers(self, seed: int, scale: float, layer_end: Sequence[int], deliveries=(), stream=None, copy_stream=None) -> None:
        """Layer-wise perturbation with the compressed coefficients of each layer arriving from the host on
        `copy_stream` while earlier layers are swept (zgr_perturb_layers).  deliveries: tuples
        (tensor, q_host, scale_host, zero_host or None[, U_host or None]) of host tensors (pinned for overlap);
        q_host / scale_host may be None when only a subspace travels."""
        nl, nd = len(layer_end), len(deliveries)
        arr = (ZgrCoeffDelivery * max(nd, 1))()
        for i, d in enumerate(deliveries):
            l, q, sc, ze = d[:4]
            U = d[4] if len(d) > 4 else None
            for h in (q, sc, ze, U):
                assert h is None or (not h.is_cuda and h.is_contiguous())
            arr[i] = ZgrCoeffDelivery(l, None if q is None else q.data_ptr(), None if sc is None else sc.data_ptr(),
                                      None if ze is None else ze.data_ptr(), None if U is None else U.data_ptr())
        self._keep.append(list(deliveries))
        if copy_stream is None:
            import torch
            copy_stream = torch.cuda.current_stream()
        _check(lib().zgr_perturb_layers(self._h, seed, scale, nl, (ctypes.c_int32 * nl)(*layer_end), nd, arr, _stream_ptr(stream),
                                        ctypes.c_void_p(copy_stream.cuda_stream)), "zgr_perturb_layers")

    def clear_coeffs(self, tensor: int) -> None:
        _check(lib().zgr_clear_coeffs(self._h, tensor), "zgr_clear_coeffs")

    def update_subspace(self, tensor: int, U_src=None, stream=None) -> None:
        """New subspace for `tensor`: a torch tensor on the host (pinned for an asynchronous copy) or on
        the device, or None if the device buffer given at construction was rewritten in place."""
        if U_src is None:
            ptr, host = None, 0
        else:
            assert U_src.is_contiguous() and U_src.dtype == self._keep[1][tensor].dtype and U_src.shape == self._keep[1][tensor].shape
            ptr, host = U_src.data_ptr(), 0 if U_src.is_cuda else 1
        _check(lib().zgr_update_subspace(self._h, tensor, ptr, host, _stream_ptr(stream)), "zgr_update_subspace")

    def update_subspaces(self, tensors: Sequence[int], U_srcs: Sequence, stream=None) -> None:
        """New subspaces for several tensors in one call (zgr_update_subspaces); all sources on the host
        (pinned for asynchronous copies) or all on the device, None for a buffer rewritten in place."""
        n = len(tensors)
        assert n == len(U_srcs) and n > 0
        host = None
        ptrs = (ctypes.c_void_p * n)()
        for i, (l, U) in enumerate(zip(tensors, U_srcs)):
            if U is None:
                ptrs[i] = None
                continue
            assert U.is_contiguous() and U.dtype == self._keep[1][l].dtype and U.shape == self._keep[1][l].shape
            assert host is None or host == (not U.is_cuda), "sources must be all on the host or all on the device"
            host = not U.is_cuda
            ptrs[i] = U.data_ptr()
        _check(lib().zgr_update_subspaces(self._h, n, (ctypes.c_int32 * n)(*tensors), ptrs, 1 if host else 0, _stream_ptr(stream)),
               "zgr_update_subspaces")

    def profile(self, enable: bool) -> None:
        _check(lib().zgr_profile(self._h, 1 if enable else 0), "zgr_profile")

    def profile_read(self):
        arr = (ZgrKernelTime * 64)()
        n = ctypes.c_int32()
        _check(lib().zgr_profile_read(self._h, arr, 64, ctypes.byref(n)), "zgr_profile_read")
        return [{"path": PATH_NAMES.get(e.path, str(e.path)), "dtype": e.dtype, "kpad": e.kpad, "launches": e.launches,
                 "elements": e.elements, "ms_total": e.ms_total} for e in arr[: n.value]]

    def enable_stats(self, on: bool) -> None:
        """Keep the norm bookkeeping inside the first perturbation of every seed (zgr_enable_stats)."""
        _check(lib().zgr_enable_stats(self._h, 1 if on else 0), "zgr_enable_stats")

    # -- bookkeeping and test hooks -------------------------------------------------------------
    def get_stats(self, seed: int, stream=None):
        import numpy as np
        out = (ctypes.c_double * (3 * self.n))()
        _check(lib().zgr_get_stats(self._h, seed, out, _stream_ptr(stream)), "zgr_get_stats")
        return np.ctypeslib.as_array(out).reshape(self.n, 3).copy()

    def tensor_norms_noalloc(self, seed: int, tensor: int, out, stream=None) -> None:
        """Norms of one tensor into `out` (a CUDA tensor of 3 float64) without any allocation by the
        library; asynchronous on the stream.  See zgr_tensor_norms_noalloc in zgr.h for the limits."""
        _check(lib().zgr_tensor_norms_noalloc(self._h, seed, tensor, out.data_ptr(), _stream_ptr(stream)), "zgr_tensor_norms_noalloc")

    def debug_philox(self, seed: int, tensor: int, tag: int, first_block: int, n_blocks: int, stream=None):
        import torch
        out = torch.empty((n_blocks, 4), dtype=torch.int32, device="cuda")
        _check(lib().zgr_debug_philox(self._h, seed, tensor, tag, first_block, n_blocks, out.data_ptr(), _stream_ptr(stream)), "zgr_debug_philox")
        return out

    def debug_z(self, seed: int, tensor: int, stream=None):
        import torch
        w = self._keep[0][tensor]
        out = torch.empty(w.shape, dtype=torch.float32, device=w.device)
        _check(lib().zgr_debug_z(self._h, seed, tensor, out.data_ptr(), _stream_ptr(stream)), "zgr_debug_z")
        return out

    def debug_z_tcgen05(self, seed: int, tensor: int, stream=None):
        """z of `tensor` in fp32 as the tcgen05 sweep kernel itself computes it (zgr_debug_z_tcgen05)."""
        import torch
        w = self._keep[0][tensor]
        out = torch.empty(w.shape, dtype=torch.float32, device=w.device)
        _check(lib().zgr_debug_z_tcgen05(self._h, seed, tensor, out.data_ptr(), _stream_ptr(stream)), "zgr_debug_z_tcgen05")
        return out

    def device_status(self) -> int:
        """Synchronise and return the device-side status code (0 = healthy)."""
        code = ctypes.c_int32()
        _check(lib().zgr_device_status(self._h, ctypes.byref(code)), "zgr_device_status")
        return code.value

    def scalars(self):
        a, b = ctypes.c_double(), ctypes.c_double()
        _check(lib().zgr_get_scalars(self._h, ctypes.byref(a), ctypes.byref(b)), "zgr_get_scalars")
        return a.value, b.value

    def state(self):
        act, seed, net = ctypes.c_int32(), ctypes.c_uint64(), ctypes.c_double()
        _check(lib().zgr_get_state(self._h, ctypes.byref(act), ctypes.byref(seed), ctypes.byref(net)), "zgr_get_state")
        return bool(act.value), seed.value, net.value

    def active_seeds(self) -> int:
        """Number of seeds whose perturbation is currently applied to the weights."""
        act, seed, net = ctypes.c_int32(), ctypes.c_uint64(), ctypes.c_double()
        _check(lib().zgr_get_state(self._h, ctypes.byref(act), ctypes.byref(seed), ctypes.byref(net)), "zgr_get_state")
        return act.value

    def launch_count(self) -> int:
        return int(lib().zgr_launch_count(self._h))

    def close(self) -> None:
        if self._h:
            lib().zgr_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def from_device_model(dm, bits_per_normal: int = 32) -> Zgr:
    """Context over a :class:`synth.DeviceModel`, with its DTC payloads attached if it has any."""
    wl = dm.workload
    z = Zgr(dm.theta, dm.U, wl.alpha, wl.eps, wl.scale_mode, bits_per_normal)
    if wl.dtc:
        for l, q in enumerate(dm.q):
            if q is not None:
                z.set_coeffs_dtc(l, q, dm.scale[l])
    return z
