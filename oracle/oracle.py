"""ctypes front end of the CPU oracle -- TEST INFRASTRUCTURE ONLY.

Runs a chain of layout operators the slow, literal way: one naive loop nest
and one fully materialised intermediate tensor per operator, in order
(Section 2.1 of the paper describes each such operator as a load/store pair in
a loop nest; equations (1) and (2) claim the composed access reads the same
values, which is what the CUDA library is checked against).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "layout_oracle.c")
_LIB = os.path.join(_HERE, "liblayout_oracle.so")
_lib = None

_i64p = ctypes.POINTER(ctypes.c_int64)
_i32p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile layout_oracle.c with gcc (idempotent)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _i64(a):
    arr = (ctypes.c_int64 * len(a))(*[int(v) for v in a])
    return arr


def _i32(a):
    return (ctypes.c_int32 * len(a))(*[int(v) for v in a])


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _check(rc, what):
    if rc != 0:
        raise ValueError("oracle %s refused its arguments (code %d)" % (what, rc))


def _raw(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype.kind not in "u":
        a = a.view({1: np.uint8, 2: np.uint16, 4: np.uint32, 8: np.uint64}[a.dtype.itemsize])
    return a


# ---------------------------------------------------------------------------
# single operators (each returns a new array; shapes inferred here)
# ---------------------------------------------------------------------------
def reshape(x, shape, nt=1):
    x = _raw(x)
    shape = [int(s) for s in shape]
    out = np.empty(shape, dtype=x.dtype)
    _check(
        lib().oracle_reshape(_ptr(x), _ptr(out), x.ndim, _i64(x.shape), len(shape), _i64(shape), x.itemsize, nt),
        "reshape",
    )
    return out


def transpose(x, perm, nt=1):
    x = _raw(x)
    if len(perm) != x.ndim:
        raise ValueError("perm rank")
    out = np.empty([x.shape[p] for p in perm], dtype=x.dtype)
    _check(lib().oracle_transpose(_ptr(x), _ptr(out), x.ndim, _i64(x.shape), _i32(perm), x.itemsize, nt), "transpose")
    return out


def slice_(x, start, stop, step, nt=1):
    x = _raw(x)
    out_shape = [-(-(int(b) - int(a)) // int(s)) for a, b, s in zip(start, stop, step)]
    out = np.empty(out_shape, dtype=x.dtype)
    _check(
        lib().oracle_slice(_ptr(x), _ptr(out), x.ndim, _i64(x.shape), _i64(start), _i64(stop), _i64(step), x.itemsize, nt),
        "slice",
    )
    return out


def concat(xs, axis, nt=1):
    xs = [_raw(x) for x in xs]
    rank = xs[0].ndim
    for x in xs:
        if x.ndim != rank or x.dtype != xs[0].dtype:
            raise ValueError("concat inputs differ in rank or type")
        if any(x.shape[d] != xs[0].shape[d] for d in range(rank) if d != axis):
            raise ValueError("concat inputs differ off the axis")
    out_shape = list(xs[0].shape)
    out_shape[axis] = sum(x.shape[axis] for x in xs)
    out = np.empty(out_shape, dtype=xs[0].dtype)
    ptrs = (ctypes.c_void_p * len(xs))(*[x.ctypes.data for x in xs])
    _check(
        lib().oracle_concat(
            len(xs), ptrs, _i64([x.shape[axis] for x in xs]), _ptr(out), rank, _i64(xs[0].shape), axis, xs[0].itemsize, nt
        ),
        "concat",
    )
    return out


def pad(x, lo, hi, nt=1):
    x = _raw(x)
    out = np.empty([a + n + b for a, n, b in zip(lo, x.shape, hi)], dtype=x.dtype)
    _check(lib().oracle_pad(_ptr(x), _ptr(out), x.ndim, _i64(x.shape), _i64(lo), _i64(hi), x.itemsize, nt), "pad")
    return out


def window(x, kh, kw, stride, padding, nt=1, dilation=1, order="rsc"):
    """NHWC im2col = zero pad on H and W, then the window gather: two operators.  `order`: "rsc" (column
    (r*kw+s)*C+c) or "crs" (column (c*kh+r)*kw+s); taps are `dilation` pixels apart."""
    x = _raw(x)
    if x.ndim != 4:
        raise ValueError("window wants NHWC")
    if order not in ("rsc", "crs"):
        raise ValueError("window column order")
    xp = pad(x, [0, padding, padding, 0], [0, padding, padding, 0], nt)
    N, Hp, Wp, C = xp.shape
    if dilation == 1 and order == "rsc":
        Ho, Wo = (Hp - kh) // stride + 1, (Wp - kw) // stride + 1
        out = np.empty([N * Ho * Wo, kh * kw * C], dtype=x.dtype)
        _check(lib().oracle_window_gather(_ptr(xp), _ptr(out), _i64(xp.shape), kh, kw, stride, x.itemsize, nt), "window")
        return out
    Ho = (Hp - dilation * (kh - 1) - 1) // stride + 1
    Wo = (Wp - dilation * (kw - 1) - 1) // stride + 1
    out = np.empty([N * Ho * Wo, kh * kw * C], dtype=x.dtype)
    _check(
        lib().oracle_window_gather_ex(
            _ptr(xp), _ptr(out), _i64(xp.shape), ctypes.c_int64(kh), ctypes.c_int64(kw), ctypes.c_int64(stride),
            ctypes.c_int64(dilation), int(order == "crs"), x.itemsize, nt,
        ),
        "window",
    )
    return out


def tile(x, reps, nt=1):
    x = _raw(x)
    if len(reps) != x.ndim:
        raise ValueError("reps rank")
    out = np.empty([int(r) * n for r, n in zip(reps, x.shape)], dtype=x.dtype)
    _check(lib().oracle_tile(_ptr(x), _ptr(out), x.ndim, _i64(x.shape), _i64(reps), x.itemsize, nt), "tile")
    return out


def repeat(x, axis, count, nt=1):
    x = _raw(x)
    shape = list(x.shape)
    shape[axis] *= int(count)
    out = np.empty(shape, dtype=x.dtype)
    _check(
        lib().oracle_repeat(_ptr(x), _ptr(out), x.ndim, _i64(x.shape), int(axis), ctypes.c_int64(int(count)), x.itemsize, nt),
        "repeat",
    )
    return out


def split_part(x, axis, sizes, part, nt=1):
    """Part number `part` of x cut along `axis` into consecutive parts of the given sizes."""
    x = _raw(x)
    shape = list(x.shape)
    shape[axis] = int(sizes[part])
    out = np.empty(shape, dtype=x.dtype)
    _check(
        lib().oracle_split_part(
            _ptr(x), _ptr(out), x.ndim, _i64(x.shape), int(axis), len(sizes), _i64(sizes), int(part), x.itemsize, nt
        ),
        "split",
    )
    return out


def affine_stmt(dst, bounds, load, store, guarded=False, fill=0):
    """Run one load/store pair in the paper's form in place on `dst`.

    load = None (store the constant) or (src array, C rows, b); store = (C rows, b).
    """
    dst_raw = _raw(dst)
    assert dst_raw.ctypes.data == dst.ctypes.data, "dst must be contiguous"
    n = len(bounds)
    es = dst_raw.itemsize
    fill_bytes = (ctypes.c_ubyte * 16)(*int(fill).to_bytes(16, "little"))
    Cs, bs = store
    Cs_flat = [v for row in Cs for v in row] or [0]
    if load is None:
        rc = lib().oracle_affine_stmt(
            None, 0, None, None, None, _ptr(dst_raw), dst_raw.ndim, _i64(dst_raw.shape), _i64(Cs_flat), _i64(bs),
            n, _i64(bounds or [0]), 0, fill_bytes, es,
        )
    else:
        src, Cl, bl = load
        src = _raw(src)
        Cl_flat = [v for row in Cl for v in row] or [0]
        rc = lib().oracle_affine_stmt(
            _ptr(src), src.ndim, _i64(src.shape), _i64(Cl_flat), _i64(bl), _ptr(dst_raw), dst_raw.ndim,
            _i64(dst_raw.shape), _i64(Cs_flat), _i64(bs), n, _i64(bounds or [0]), int(bool(guarded)), fill_bytes, es,
        )
    _check(rc, "affine_stmt")
    return dst


# ---------------------------------------------------------------------------
# a whole chain, operator by operator
# ---------------------------------------------------------------------------
def run_chain(chain, inputs, nt=1, keep_intermediates=False):
    """Execute `chain` (paper_2002_12798_b200.workloads.Chain-like object with
    .inputs and .ops) on `inputs` sequentially.  Returns the output array, or
    the list of all tensors when keep_intermediates is set."""
    tensors = [_raw(x) for x in inputs]
    if len(tensors) != len(chain.inputs):
        raise ValueError("wrong number of inputs")
    for op in chain.ops:
        kind = op["kind"]
        if kind == "reshape":
            t = reshape(tensors[op["src"]], op["shape"], nt)
        elif kind == "transpose":
            t = transpose(tensors[op["src"]], op["perm"], nt)
        elif kind == "slice":
            t = slice_(tensors[op["src"]], op["start"], op["stop"], op["step"], nt)
        elif kind == "concat":
            t = concat([tensors[s] for s in op["srcs"]], op["axis"], nt)
        elif kind == "pad":
            t = pad(tensors[op["src"]], op["lo"], op["hi"], nt)
        elif kind == "window":
            t = window(tensors[op["src"]], op["kh"], op["kw"], op["stride"], op["pad"], nt, op.get("dilation", 1),
                       op.get("order", "rsc"))
        elif kind == "tile":
            t = tile(tensors[op["src"]], op["reps"], nt)
        elif kind == "repeat":
            t = repeat(tensors[op["src"]], op["axis"], op["count"], nt)
        elif kind == "split":
            t = split_part(tensors[op["src"]], op["axis"], op["sizes"], op["part"], nt)
        elif kind == "stmts":
            # elements no statement writes stay at a recognisable poison value
            t = np.full(op["shape"], 0xA5, dtype=np.uint8).astype(tensors[0].dtype)
            t[...] = np.frombuffer(b"\xa5" * t.itemsize, dtype=t.dtype)[0]
            for st in op["stmts"]:
                load = None
                if st["load"] is not None:
                    lt, Cl, bl = st["load"]
                    load = (tensors[lt], Cl, bl)
                affine_stmt(t, st["bounds"], load, st["store"], st.get("guarded", False), st.get("fill", 0))
        else:
            raise ValueError("unknown operator kind %r" % kind)
        tensors.append(t)
    return tensors if keep_intermediates else tensors[-1]
