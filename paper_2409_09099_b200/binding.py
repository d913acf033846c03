"""Thin ctypes binding of libsste: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors used purely as device memory (``data_ptr()``);
every computation runs in the library's kernels on torch's current stream.
There is no fallback: if the shared library is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_HERE = Path(__file__).resolve().parent
LIB_PATH = _HERE / "libsste.so"

BF16, F32, E4M3, E5M2 = 0, 1, 2, 3
PRUNE_SOFT, PRUNE_HARD = 0, 1
OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_DTYPE, ERR_ALIGN, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA, ERR_DEGENERATE, \
    ERR_TIMEOUT = range(10)

_TORCH_DT = {BF16: torch.bfloat16, F32: torch.float32, E4M3: torch.float8_e4m3fn, E5M2: torch.float8_e5m2}
_CODE_OF = {v: k for k, v in _TORCH_DT.items()}

EXPORTS = [
    "sste_workspace_bytes", "sste_create", "sste_destroy", "sste_status_string", "sste_poll_device_status",
    "sste_vals_bytes", "sste_meta_bytes", "sste_beta_init", "sste_project_compress", "sste_linear_fwd",
    "sste_mvue_sparsify", "sste_linear_bwd_input", "sste_linear_bwd_weight", "sste_amax", "sste_fp8_scale",
    "sste_quantize_fp8", "sste_meta_to_canonical", "sste_debug_force_tile_width", "sste_debug_force_splits",
    "sste_workspace_bytes_recommended", "sste_beta_init_static", "sste_debug_launch_count", "sste_flip_count",
    "sste_project_compress_variant", "sste_beta_init_l1", "sste_srste_decay", "sste_project_amax",
    "sste_decompress", "sste_padded_dim", "sste_pad_2d", "sste_crop_2d", "sste_debug_inject_stall",
    "sste_debug_force_tile_order", "sste_debug_plan", "sste_debug_tile_coords",
    "sste_debug_mvue_groups", "sste_debug_selftest_device_once",
]


class SsteError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"libsste: {what} (status {code})")
        self.code = code


_lib = None


def load() -> ctypes.CDLL:
    """Load libsste.so from the package directory (built by ``build.py``); raises if absent."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise FileNotFoundError(f"{LIB_PATH} not built: run python -m paper_2409_09099_b200.build")
        lib = ctypes.CDLL(str(LIB_PATH))
        lib.sste_workspace_bytes.restype = ctypes.c_size_t
        lib.sste_workspace_bytes_recommended.restype = ctypes.c_size_t
        lib.sste_vals_bytes.restype = ctypes.c_size_t
        lib.sste_meta_bytes.restype = ctypes.c_size_t
        lib.sste_status_string.restype = ctypes.c_char_p
        _lib = lib
    return _lib


def _ptr(t):
    if t is None:
        return ctypes.c_void_p(0)
    assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def padded_dim(n: int) -> int:
    """sste_padded_dim: the next multiple of 128."""
    return int(load().sste_padded_dim(n))


def plan(product: int, opdt: int, O: int, I: int, T: int, sm_count: int = 148, workspace_bytes: int | None = None):
    """sste_debug_plan: (tile width, split-K factor, first split tile, band height) of a product launch; host only."""
    lib = load()
    ws = lib.sste_workspace_bytes_recommended() if workspace_bytes is None else workspace_bytes
    out = [ctypes.c_int() for _ in range(4)]
    st = lib.sste_debug_plan(product, opdt, O, I, T, sm_count, ctypes.c_size_t(ws), *[ctypes.byref(o) for o in out])
    if st != OK:
        raise SsteError(st, lib.sste_status_string(st).decode())
    return tuple(o.value for o in out)


def launch_count() -> int:
    """Kernels launched by the library in this process so far (sste_debug_launch_count)."""
    lib = load()
    lib.sste_debug_launch_count.restype = ctypes.c_ulonglong
    return int(lib.sste_debug_launch_count())


def beta_init_static(W, beta_dev):
    """sste_beta_init_static: beta for callers that cannot lend a device workspace.

    Needs no Context and allocates nothing on the device: the reduction scratch is a fixed array inside
    libsste.so.  Same arguments as Context.beta_init; W may have at most 8192 tiles of 128 x 128.
    Raises SsteError (code ERR_WORKSPACE for a tensor beyond that limit).
    """
    lib = load()
    O, I = W.shape
    st = lib.sste_beta_init_static(W.device.index or 0, _ptr(W), O, I, _CODE_OF[W.dtype], _ptr(beta_dev), _stream())
    if st != OK:
        raise SsteError(st, lib.sste_status_string(st).decode())


class Context:
    """Owns the device workspace (a torch allocation) and the sste_ctx handle."""

    def __init__(self, device: int = 0, minimal_workspace: bool = False):
        self.lib = load()
        self.device = device
        n = self.lib.sste_workspace_bytes() if minimal_workspace else self.lib.sste_workspace_bytes_recommended()
        self.workspace = torch.zeros(n, dtype=torch.uint8, device=f"cuda:{device}")
        handle = ctypes.c_void_p()
        st = self.lib.sste_create(ctypes.byref(handle), device, _ptr(self.workspace), ctypes.c_size_t(n))
        self._check(st)
        self.handle = handle

    def close(self):
        if getattr(self, "handle", None):
            self.lib.sste_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != OK:
            raise SsteError(st, self.lib.sste_status_string(st).decode())

    # ---- hot path -------------------------------------------------------------------------------

    def beta_init(self, W, beta_dev):
        O, I = W.shape
        self._check(self.lib.sste_beta_init(self.handle, _ptr(W), O, I, _CODE_OF[W.dtype], _ptr(beta_dev), _stream()))

    def project_compress(self, W, beta_dev, vals, meta, dense_out=None, w_amax_dev=None):
        O, I = W.shape
        self._check(self.lib.sste_project_compress(
            self.handle, _ptr(W), O, I, _CODE_OF[W.dtype], _ptr(beta_dev), _ptr(w_amax_dev), _CODE_OF[vals.dtype],
            _ptr(vals), _ptr(meta), _ptr(dense_out), _stream()))

    def linear_fwd(self, X, vals, meta, Y, x_amax_dev=None, w_amax_dev=None, y_amax_out_dev=None):
        T, I = X.shape
        O = vals.shape[0]
        self._check(self.lib.sste_linear_fwd(
            self.handle, _ptr(X), T, _ptr(vals), _ptr(meta), O, I, _CODE_OF[X.dtype], _ptr(x_amax_dev),
            _ptr(w_amax_dev), _ptr(Y), _CODE_OF[Y.dtype], _ptr(y_amax_out_dev), _stream()))

    def mvue_sparsify(self, dY, seed, tensor_id, step, gvals, gmeta, dense_q_out=None, g_amax_dev=None,
                      token_offset=0, counter_cols=0):
        T, O = dY.shape
        self._check(self.lib.sste_mvue_sparsify(
            self.handle, _ptr(dY), T, O, _CODE_OF[dY.dtype], ctypes.c_uint64(seed), ctypes.c_uint32(tensor_id),
            ctypes.c_uint32(step), ctypes.c_uint64(token_offset), ctypes.c_int(counter_cols), _ptr(g_amax_dev),
            _CODE_OF[gvals.dtype], _ptr(gvals), _ptr(gmeta), _ptr(dense_q_out), _stream()))

    def linear_bwd_input(self, dY, Wt_dense, dX, g_amax_dev=None, w_amax_dev=None, vals=None, meta=None,
                         dx_amax_out_dev=None):
        """grad_X from the dense copy `Wt_dense`, or (Wt_dense=None) from the compressed operand (vals, meta)."""
        T, O = dY.shape
        if Wt_dense is not None:
            I, wdt = Wt_dense.shape[1], _CODE_OF[Wt_dense.dtype]
        else:
            I, wdt = 2 * vals.shape[1], _CODE_OF[vals.dtype]
        self._check(self.lib.sste_linear_bwd_input(
            self.handle, _ptr(dY), T, O, _CODE_OF[dY.dtype], _ptr(Wt_dense), _ptr(vals), _ptr(meta), I, wdt,
            _ptr(g_amax_dev), _ptr(w_amax_dev), _ptr(dX), _CODE_OF[dX.dtype], _ptr(dx_amax_out_dev), _stream()))

    def linear_bwd_weight(self, gvals, gmeta, X, dW, g_amax_dev=None, x_amax_dev=None):
        O = gvals.shape[0]
        T, I = X.shape
        self._check(self.lib.sste_linear_bwd_weight(
            self.handle, _ptr(gvals), _ptr(gmeta), O, T, _CODE_OF[gvals.dtype], _ptr(X), I, _CODE_OF[X.dtype],
            _ptr(g_amax_dev), _ptr(x_amax_dev), _ptr(dW), _CODE_OF[dW.dtype], _stream()))

    # ---- FP8 helpers ----------------------------------------------------------------------------

    def amax(self, x, amax_dev):
        self._check(self.lib.sste_amax(self.handle, _ptr(x), ctypes.c_size_t(x.numel()), _CODE_OF[x.dtype],
                                       _ptr(amax_dev), _stream()))

    def project_amax(self, W, beta_dev, amax_dev):
        O, I = W.shape
        self._check(self.lib.sste_project_amax(self.handle, _ptr(W), O, I, _CODE_OF[W.dtype], _ptr(beta_dev),
                                               _ptr(amax_dev), _stream()))

    def fp8_scale(self, amax_dev, odt, scale_dev, inv_scale_dev=None):
        self._check(self.lib.sste_fp8_scale(self.handle, _ptr(amax_dev), odt, _ptr(scale_dev), _ptr(inv_scale_dev),
                                            _stream()))

    def quantize_fp8(self, x, amax_dev, q):
        self._check(self.lib.sste_quantize_fp8(self.handle, _ptr(x), ctypes.c_size_t(x.numel()), _ptr(amax_dev),
                                               _CODE_OF[q.dtype], _ptr(q), _stream()))

    # ---- ablation variants of the pruning step ---------------------------------------------------

    def project_compress_variant(self, W, beta_dev, vals, meta, dense_out=None, w_amax_dev=None, hard=False,
                                 gamma=0.0):
        O, I = W.shape
        self._check(self.lib.sste_project_compress_variant(
            self.handle, _ptr(W), O, I, _CODE_OF[W.dtype], _ptr(beta_dev), _ptr(w_amax_dev), _CODE_OF[vals.dtype],
            PRUNE_HARD if hard else PRUNE_SOFT, ctypes.c_float(gamma), _ptr(vals), _ptr(meta), _ptr(dense_out),
            _stream()))

    def beta_init_l1(self, W, beta_dev):
        O, I = W.shape
        self._check(self.lib.sste_beta_init_l1(self.handle, _ptr(W), O, I, _CODE_OF[W.dtype], _ptr(beta_dev),
                                               _stream()))

    def srste_decay(self, W, meta, meta_dt, lam, dW):
        O, I = W.shape
        self._check(self.lib.sste_srste_decay(self.handle, _ptr(W), _ptr(meta), O, I, meta_dt, ctypes.c_float(lam),
                                              _ptr(dW), _stream()))

    # ---- diagnostics ----------------------------------------------------------------------------

    def flip_count(self, meta_prev, meta_cur, rows, k, count_dev):
        """sste_flip_count: mask entries that changed between two metadata images of a [rows, k] weight."""
        self._check(self.lib.sste_flip_count(self.handle, _ptr(meta_prev), _ptr(meta_cur), rows, k, _ptr(count_dev),
                                             _stream()))

    # ---- helpers --------------------------------------------------------------------------------

    def decompress(self, vals, meta, dense_out):
        rows, k = dense_out.shape
        self._check(self.lib.sste_decompress(self.handle, _ptr(vals), _ptr(meta), rows, k, _CODE_OF[vals.dtype],
                                             _ptr(dense_out), _stream()))

    def pad_2d(self, src, dst):
        """dst[:rows, :cols] = src, zeros elsewhere (2-byte elements)."""
        self._check(self.lib.sste_pad_2d(self.handle, _ptr(src), src.shape[0], src.shape[1], _ptr(dst), dst.shape[0],
                                         dst.shape[1], _stream()))

    def crop_2d(self, src, dst):
        """dst = src[:rows, :cols] (2-byte elements)."""
        self._check(self.lib.sste_crop_2d(self.handle, _ptr(src), src.shape[0], src.shape[1], _ptr(dst), dst.shape[0],
                                          dst.shape[1], _stream()))

    def meta_to_canonical(self, meta, rows, k, dt, out):
        self._check(self.lib.sste_meta_to_canonical(self.handle, _ptr(meta), rows, k, dt, _ptr(out), _stream()))

    def debug_mvue_groups(self, a, k24, pos_out, val_out):
        """sste_debug_mvue_groups: the MVUE group rule on explicit groups a [n, 4] (bf16) and 24-bit uniforms k24 [n]."""
        self._check(self.lib.sste_debug_mvue_groups(self.handle, _ptr(a), _ptr(k24), ctypes.c_size_t(a.shape[0]),
                                                    _ptr(pos_out), _ptr(val_out), _stream()))

    def debug_force_splits(self, splits: int):
        self._check(self.lib.sste_debug_force_splits(splits))

    def debug_force_tile_order(self, group_m: int):
        self._check(self.lib.sste_debug_force_tile_order(group_m))

    def debug_inject_stall(self, on: bool):
        self._check(self.lib.sste_debug_inject_stall(1 if on else 0))

    def debug_force_tile_width(self, bn: int):
        self._check(self.lib.sste_debug_force_tile_width(bn))

    def poll_device_status(self) -> int:
        return self.lib.sste_poll_device_status(self.handle, _stream())

    # ---- allocation helpers (torch as the allocator) ---------------------------------------------

    def alloc_compressed(self, rows, k, dt=BF16):
        dev = f"cuda:{self.device}"
        vals = torch.empty((rows, k // 2), dtype=_TORCH_DT[dt], device=dev)
        meta = torch.empty(self.lib.sste_meta_bytes(rows, k), dtype=torch.uint8, device=dev)
        return vals, meta
