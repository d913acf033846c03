"""S-STE oracle, Python face.  TEST INFRASTRUCTURE ONLY.

A plain CPU statement of the sparse linear layer's hot path, written from the
paper: the elementwise parts are the C file next to this one (compiled with gcc,
no FMA contraction), the three matrix products are numpy fp64 matmuls on the
decoded operands.  Nothing here imports, loads or shares code with the CUDA
library; only tests, the smoke check and the bench's CPU-baseline leg may use it.

Arrays: bf16 tensors are numpy uint16 bit patterns, fp8 tensors uint8 bit
patterns.  dtype codes: 0 = bf16, 2 = E4M3, 3 = E5M2.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "sste_oracle.c"
_LIB = _HERE / "libsste_oracle.so"

BF16, F32, E4M3, E5M2 = 0, 1, 2, 3
FP8_MAX = {E4M3: 448.0, E5M2: 57344.0}


def build(force: bool = False) -> Path:
    """Compile the C oracle (gcc, -ffp-contract=off so fp32 steps are single IEEE ops)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
             str(_SRC), "-o", str(tmp), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.sste_oracle_beta.restype = ctypes.c_double
        _lib.sste_oracle_amax_bf16.restype = ctypes.c_float
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dt):
    a = np.ascontiguousarray(a)
    assert a.dtype == dt, (a.dtype, dt)
    return a


# ----------------------------------------------------------------- codecs

def bf16_to_f32(x):
    x = _c(x, np.uint16)
    out = np.empty(x.shape, np.float32)
    lib().sste_oracle_bf16_to_f32(_p(x), ctypes.c_int64(x.size), _p(out))
    return out


def f32_to_bf16(x):
    x = _c(x, np.float32)
    out = np.empty(x.shape, np.uint16)
    lib().sste_oracle_f32_to_bf16(_p(x), ctypes.c_int64(x.size), _p(out))
    return out


def f32_to_fp8(x, odt):
    x = _c(x, np.float32)
    out = np.empty(x.shape, np.uint8)
    lib().sste_oracle_f32_to_fp8(_p(x), ctypes.c_int64(x.size), ctypes.c_int(odt), _p(out))
    return out


def fp8_to_f32(x, dt):
    x = _c(x, np.uint8)
    out = np.empty(x.shape, np.float32)
    lib().sste_oracle_fp8_to_f32(_p(x), ctypes.c_int64(x.size), ctypes.c_int(dt), _p(out))
    return out


def decode(x, dt):
    """bit patterns -> float64 values"""
    if dt == BF16:
        return bf16_to_f32(x).astype(np.float64)
    return fp8_to_f32(x, dt).astype(np.float64)


# ----------------------------------------------- projection, beta, compress

def s_soft(W):
    """Eq. (4): 2:4 soft-thresholding of a bf16 [O, I] matrix, groups along I; fp32 result."""
    W = _c(W, np.uint16)
    O, I = W.shape
    assert I % 4 == 0
    S = np.empty((O, I), np.float32)
    lib().sste_oracle_s_soft(_p(W), O, I, _p(S))
    return S


def beta(W):
    """Eq. (5): beta = <w, S_soft(w)> / ||S_soft(w)||^2 in fp64.  Returns (beta, num, den, degenerate)."""
    W = _c(W, np.uint16)
    O, I = W.shape
    num, den, deg = ctypes.c_double(), ctypes.c_double(), ctypes.c_int()
    b = lib().sste_oracle_beta(_p(W), O, I, ctypes.byref(num), ctypes.byref(den), ctypes.byref(deg))
    return b, num.value, den.value, bool(deg.value)


def project_compress(W, beta32, odt=BF16, wscale=1.0, want_dense=True):
    """w~ = cast(fl32(S_soft(w) * beta) [* wscale]) compressed to canonical (vals, meta) [+ dense w~]."""
    W = _c(W, np.uint16)
    O, I = W.shape
    assert I % 16 == 0
    vdt = np.uint16 if odt == BF16 else np.uint8
    vals = np.empty((O, I // 2), vdt)
    meta = np.zeros((O, I // 16), np.uint16)
    dense = np.empty((O, I), vdt) if want_dense else None
    lib().sste_oracle_project_compress(_p(W), O, I, ctypes.c_float(beta32), ctypes.c_float(wscale),
                                       ctypes.c_int(odt), _p(vals), _p(meta), _p(dense))
    return vals, meta, dense


def decompress(vals, meta, dt=BF16):
    """canonical (vals [rows, K/2], meta [rows, K/16]) -> dense fp32 [rows, K]"""
    rows, K2 = vals.shape
    K = 2 * K2
    vals = _c(vals, np.uint16 if dt == BF16 else np.uint8)
    meta = _c(meta, np.uint16)
    dense = np.empty((rows, K), np.float32)
    lib().sste_oracle_decompress(_p(vals), _p(meta), rows, K, ctypes.c_int(dt), _p(dense))
    return dense


# ------------------------------------------------------------ Philox, MVUE

def philox4x32_10(ctr, key):
    ctr = np.asarray(ctr, np.uint32).copy()
    key = np.asarray(key, np.uint32).copy()
    out = np.empty(4, np.uint32)
    lib().sste_oracle_philox4x32_10(_p(ctr), _p(key), _p(out))
    return out


def mvue_group(a, u):
    """One group of 4 (fp32) and one uniform u: returns (positions[2], values[2])."""
    a = np.asarray(a, np.float32).copy()
    pos = np.empty(2, np.int32)
    val = np.empty(2, np.float32)
    lib().sste_oracle_mvue_group(_p(a), ctypes.c_float(u), _p(pos), _p(val))
    return pos, val


def mvue(dY, seed, tensor_id, step, odt=BF16, gscale=1.0, want_dense_q=False, want_theta=False, token_offset=0):
    """MVUE(dY^T) of a bf16 [T, O] gradient: canonical compressed [O, T/2] + meta [O, T/16].

    token_offset: tokens that precede this dY in the whole batch (the counter is the global group index).
    """
    assert token_offset % 4 == 0
    dY = _c(dY, np.uint16)
    T, O = dY.shape
    assert T % 16 == 0
    vdt = np.uint16 if odt == BF16 else np.uint8
    gvals = np.empty((O, T // 2), vdt)
    gmeta = np.zeros((O, T // 16), np.uint16)
    dense_q = np.empty((T, O), np.uint8) if want_dense_q else None
    theta = np.empty((T, O), np.float32) if want_theta else None
    lib().sste_oracle_mvue(_p(dY), T, O, ctypes.c_uint64(seed), ctypes.c_uint32(tensor_id),
                           ctypes.c_uint32(step), ctypes.c_uint64(token_offset // 4), ctypes.c_float(gscale),
                           ctypes.c_int(odt),
                           _p(gvals), _p(gmeta), _p(dense_q), _p(theta))
    return gvals, gmeta, dense_q, theta


# ------------------------------------------------------------ FP8 scaling

def amax(x):
    x = _c(x, np.uint16)
    return float(lib().sste_oracle_amax_bf16(_p(x), ctypes.c_int64(x.size)))


def fp8_scale(amax_value, odt):
    """Per-tensor scale = fl32(FP8_MAX / amax); 1 when amax is 0 (Sec. 5.2: rescale, then cast)."""
    if amax_value == 0.0:
        return np.float32(1.0)
    return np.float32(np.float32(FP8_MAX[odt]) / np.float32(amax_value))


def quantize(x, scale, odt):
    x = _c(x, np.uint16)
    q = np.empty(x.shape, np.uint8)
    lib().sste_oracle_quantize_bf16(_p(x), ctypes.c_int64(x.size), ctypes.c_float(scale),
                                    ctypes.c_int(odt), _p(q))
    return q


# ------------------------------------------------ the three products (Sec. 5.1)

def linear_fwd(X, xdt, vals, meta, wdt, inv_scale=1.0):
    """Z = X S(W)^T: fp64 product of the decoded operands, times inv_scale = 1/(sx*sw)."""
    Wt = decompress(vals, meta, wdt).astype(np.float64)
    return (decode(X, xdt) @ Wt.T) * inv_scale


def linear_bwd_weight(gvals, gmeta, gdt, X, xdt, inv_scale=1.0):
    """grad_W = MVUE(grad_Z^T) X: [O, T] x [T, I] in fp64."""
    G = decompress(gvals, gmeta, gdt).astype(np.float64)
    return (G @ decode(X, xdt)) * inv_scale


def linear_bwd_input(dY, gdt, Wt_dense, wdt, inv_scale=1.0):
    """grad_X = grad_Z S(W): [T, O] x [O, I] in fp64 (dense: the 2:4 structure lies along I)."""
    return (decode(dY, gdt) @ decode(Wt_dense, wdt)) * inv_scale


# ---------------------------------------------------------------- flip rate (Sec. 3.1, "Flip rate")

def hard_mask(W):
    """m_h(W): 1 where an element is one of the two largest magnitudes of its group of four.

    Ties are broken as everywhere in this oracle: magnitude descending, then index ascending.
    W: bf16 bit patterns [rows, k].  Returns uint8 [rows, k].
    """
    mag = (np.asarray(W, dtype=np.uint16) & 0x7FFF).astype(np.int64)      # bf16 magnitudes order like integers
    rows, k = mag.shape
    g = mag.reshape(rows, k // 4, 4)
    # stable sort of -magnitude keeps the lower index first among equals
    order = np.argsort(-g, axis=-1, kind="stable")
    mask = np.zeros_like(g, dtype=np.uint8)
    np.put_along_axis(mask, order[..., :2], 1, axis=-1)
    return mask.reshape(rows, k)


def flip_count(W_prev, W_cur):
    """|| m_h(W_cur) xor m_h(W_prev) ||_1 : the number of mask entries that changed between two iterations."""
    return int(np.count_nonzero(hard_mask(W_prev) != hard_mask(W_cur)))


def flip_rate(W_prev, W_cur):
    """r_k = || m_h(w_k) xor m_h(w_{k-1}) ||_1 / d  (Sec. 3.1)."""
    return flip_count(W_prev, W_cur) / float(np.asarray(W_cur).size)


# ---------------------------------------------------------------- ablation variants of the pruning step
# (Sec. 4.1 "Choosing optimal threshold", Eq. 2 hard thresholding, Sec. 4.2 "Minimizing MSE", Sec. 3.2 SR-STE)

def _groups_f32(W):
    f = bf16_to_f32(_c(W, np.uint16))
    rows, k = f.shape
    return f.reshape(rows, k // 4, 4)


def _kept_pair(mag_bits):
    """Positions of the two largest magnitudes per group: magnitude descending, index ascending."""
    order = np.argsort(-mag_bits.astype(np.int64), axis=-1, kind="stable")[..., :2]
    return np.sort(order, axis=-1)


def project_compress_variant(W, beta32, gamma=0.0, hard=False, odt=BF16, wscale=1.0):
    """The pruning step with the paper's ablation knobs; returns canonical (vals, meta, dense) like project_compress.

    hard=False: soft thresholding (Eq. 4) with the interpolated threshold t = (1 - gamma) |t2| + gamma |t3|,
    |t2| <= |t3| the second and third smallest magnitudes (Sec. 4.1: any t in [|t2|, |t3|] is feasible, gamma = 0
    gives t = |t2|, larger gamma moves t towards |t3|); fp32: t = fl(fl(fl(1 - gamma) * |t2|) + fl(gamma * |t3|)).
    hard=True: hard thresholding (Eq. 2): the two largest magnitudes are kept unchanged, the others are 0.
    Then * beta (fp32) [* wscale], one cast, compression of the kept pair.
    """
    W = _c(W, np.uint16)
    rows, k = W.shape
    a = _groups_f32(W)
    mag = np.abs(a)
    bits = (W & 0x7FFF).reshape(rows, k // 4, 4)
    pair = _kept_pair(bits)
    f32 = np.float32
    if hard:
        keep = np.zeros(a.shape, dtype=bool)
        np.put_along_axis(keep, pair, True, axis=-1)
        s = np.where(keep, a, f32(0.0))
    else:
        srt = np.sort(mag, axis=-1)
        g = f32(gamma)
        t = (f32(1.0) - g) * srt[..., 1] + g * srt[..., 2]          # every step a single fp32 operation
        t = t.astype(f32)[..., None]
        d = (a - np.copysign(t, a)).astype(f32)                      # sign(a) (|a| - t)
        s = np.where(mag > t, d, f32(0.0))
    w = (s * f32(beta32)).astype(f32)
    if odt != BF16:
        w = (w * f32(wscale)).astype(f32)
    w = np.where(s == 0, f32(0.0), w).astype(f32)                    # pruned entries are canonical +0
    enc = f32_to_bf16 if odt == BF16 else (lambda x: f32_to_fp8(x, odt))
    dense = enc(w.reshape(rows, k))
    vals = np.take_along_axis(dense.reshape(rows, k // 4, 4), pair, axis=-1).reshape(rows, k // 2)
    nib = (pair[..., 0] | (pair[..., 1] << 2)).astype(np.uint16).reshape(rows, k // 16, 4)
    meta = (nib[..., 0] | (nib[..., 1] << 4) | (nib[..., 2] << 8) | (nib[..., 3] << 12)).astype(np.uint16)
    return vals, meta, dense


def beta_l1(W):
    """The L1 rescaling the paper argues against (Sec. 4.2): beta = ||w||_1 / ||S_soft(w)||_1, fp64 sums."""
    a = _groups_f32(W).astype(np.float64)
    mag = np.abs(a)
    t = np.sort(mag, axis=-1)[..., 1:2]
    s = np.maximum(mag - t, 0.0)
    den = float(s.sum())
    return (float(mag.sum()) / den) if den > 0 else 1.0


def srste_decay(dW, W, lam):
    """Sparse-refined STE (Sec. 3.2): the gradient of (lambda / 2) ||w (1 - m_h(w))||^2 added to grad_W.

    dW, W: bf16 bit patterns [O, I]; returns bf16 bits of fl32(dW + fl32(lambda * w)) on pruned entries,
    dW unchanged on kept ones.
    """
    f32 = np.float32
    g, w = bf16_to_f32(_c(dW, np.uint16)), bf16_to_f32(_c(W, np.uint16))
    pruned = hard_mask(W) == 0
    out = np.where(pruned, (g + (f32(lam) * w).astype(f32)).astype(f32), g)
    return f32_to_bf16(out.astype(f32))
