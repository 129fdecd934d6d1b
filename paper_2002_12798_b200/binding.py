"""Thin ctypes binding of libamap.so (include/amap.h): argument marshalling only.

Every step of the path -- building statements, composing the affine maps,
planning and the copy itself -- runs inside the C/CUDA library.  PyTorch is
used only for device memory (`Tensor.data_ptr()`) and streams.  There is no
CPU fallback: if the library cannot be built or loaded, importing this module
raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_int, c_int32, c_int64, c_uint32, c_uint64, c_void_p

from . import build as _build

AMAP_CONST = -1
KERNEL_AUTO, KERNEL_GATHER, KERNEL_COPY, KERNEL_TRANSPOSE, KERNEL_FILL = 0, 1, 2, 3, 4
COMPOSE_NO_FUSE = 1
COMPOSE_QUASI_AFFINE = 2
COMPOSE_NO_QUASI_AFFINE = 4
PLAN_NO_PDL = 1
PLAN_NO_PREFETCH = 2
KERNEL_NAMES = {1: "gather", 2: "copy", 3: "transpose", 4: "fill"}
LAUNCH_NAMES = {0: "affine", 1: "strip", 2: "transpose", 3: "transpose_shifted", 4: "transpose_realign", 5: "transpose_flat", 6: "transpose_flat_source"}

EXPORTS = [
    "amap_builder_create", "amap_builder_destroy", "amap_builder_input", "amap_builder_reshape",
    "amap_builder_transpose", "amap_builder_slice", "amap_builder_concat", "amap_builder_pad",
    "amap_builder_window", "amap_builder_window_ex", "amap_builder_tile", "amap_builder_repeat", "amap_builder_split", "amap_builder_tensor",
    "amap_builder_stmt",
    "amap_builder_opaque", "amap_builder_chain", "amap_compose", "amap_compose_ex", "amap_compose_multi",
    "amap_map_num_outputs", "amap_map_output_numel", "amap_execute_multi", "amap_map_device_view", "amap_consume_row_sums", "amap_view_rows_gather_host", "amap_map_num_stages", "amap_map_get_stage", "amap_map_destroy", "amap_map_num_pieces", "amap_map_get_piece",
    "amap_map_sizes", "amap_plan", "amap_plan_destroy", "amap_plan_stats", "amap_plan_piece_kernel", "amap_plan_launch_info",
    "amap_execute", "amap_execute_host", "amap_execute_static", "amap_strerror", "amap_last_cuda_error",
]


class AmapError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        msg = _lib.amap_strerror(code).decode()
        if code == -8:
            msg += " (" + _lib.amap_last_cuda_error().decode() + ")"
        super().__init__("%s: %s [%d]" % (where, msg, code))


class _Access(Structure):
    _fields_ = [("tensor", c_int32), ("rank", c_int32), ("C", POINTER(c_int64)), ("b", POINTER(c_int64))]


class _Stmt(Structure):
    _fields_ = [
        ("n_loops", c_int32), ("bounds", POINTER(c_int64)), ("load", _Access), ("store", _Access),
        ("guarded", c_int32), ("fill_bits", c_uint64),
    ]


class _Constraint(Structure):
    _fields_ = [("coef", POINTER(c_int64)), ("offset", c_int64), ("extent", c_int64)]


class _Piece(Structure):
    _fields_ = [
        ("n_loops", c_int32), ("bounds", POINTER(c_int64)), ("input", c_int32), ("C_l", POINTER(c_int64)),
        ("b_l", c_int64), ("C_s", POINTER(c_int64)), ("b_s", c_int64), ("n_guards", c_int32),
        ("guards", POINTER(_Constraint)), ("n_domain", c_int32), ("domain", POINTER(_Constraint)),
        ("fill_bits", c_uint64), ("output", c_int32), ("n_digits", c_int32), ("digit_radix", POINTER(c_int64)),
        ("digit_stride", POINTER(c_int64)), ("F", POINTER(c_int64)), ("f0", c_int64),
    ]


VIEW_MAX_PIECES, VIEW_MAX_LOOPS, VIEW_MAX_CONS = 8, 8, 4


class _ViewCon(Structure):
    _fields_ = [("coef", c_int64 * VIEW_MAX_LOOPS), ("offset", c_int64), ("extent", c_int64)]


class _ViewPiece(Structure):
    _fields_ = [
        ("n_loops", c_int32), ("input", c_int32), ("n_guards", c_int32), ("n_domain", c_int32),
        ("ext", c_int64 * VIEW_MAX_LOOPS), ("dst_stride", c_int64 * VIEW_MAX_LOOPS), ("src_stride", c_int64 * VIEW_MAX_LOOPS),
        ("b_s", c_int64), ("b_l", c_int64), ("fill_bits", c_uint64), ("cons", _ViewCon * VIEW_MAX_CONS),
        ("fd_mul", ctypes.c_uint32 * VIEW_MAX_LOOPS), ("fd_sh1", ctypes.c_uint8 * VIEW_MAX_LOOPS),
        ("fd_sh2", ctypes.c_uint8 * VIEW_MAX_LOOPS),
    ]


class DeviceView(Structure):
    """amap_device_view (include/amap_device.h): the composed map as a plain struct a kernel takes by value."""
    _fields_ = [
        ("n_pieces", c_int32), ("elem_size", c_int32), ("n_inputs", c_int32), ("small", c_int32),
        ("out_numel", c_int64), ("piece", _ViewPiece * VIEW_MAX_PIECES),
    ]


class _PlanOpts(Structure):
    _fields_ = [("force_kernel", c_int32), ("pointer_align", c_int32), ("flags", c_int32), ("reserved", c_int32 * 5)]


class _LaunchInfo(Structure):
    _fields_ = [
        ("kernel", c_int32), ("access", c_int32), ("n_descriptors", c_int32), ("stage", c_int32),
        ("n_blocks", c_uint32), ("threads", c_int32), ("smem_bytes", c_int32), ("wide_offsets", c_int32),
    ]


class _Stats(Structure):
    _fields_ = [
        ("bytes_read", c_int64), ("bytes_written", c_int64), ("bytes_filled", c_int64), ("n_pieces", c_int32),
        ("n_launches", c_int32), ("kernel_kind", c_int32 * 4), ("n_stages", c_int32), ("n_descriptors", c_int32),
    ]


def _load():
    path = _build.build_library()
    lib = ctypes.CDLL(path)
    lib.amap_strerror.restype = c_char_p
    lib.amap_strerror.argtypes = [c_int]
    lib.amap_last_cuda_error.restype = c_char_p
    lib.amap_builder_destroy.restype = None
    lib.amap_builder_destroy.argtypes = [c_void_p]
    lib.amap_map_destroy.restype = None
    lib.amap_map_destroy.argtypes = [c_void_p]
    lib.amap_plan_destroy.restype = None
    lib.amap_plan_destroy.argtypes = [c_void_p]
    lib.amap_builder_pad.argtypes = [c_void_p, c_int32, c_int32, POINTER(c_int64), POINTER(c_int64), c_uint64, POINTER(c_int32)]
    lib.amap_execute.argtypes = [c_void_p, POINTER(c_void_p), c_void_p, c_void_p]
    lib.amap_execute_multi.argtypes = [c_void_p, POINTER(c_void_p), POINTER(c_void_p), c_void_p]
    lib.amap_execute_host.argtypes = [c_void_p, POINTER(c_void_p), c_void_p, c_void_p]
    lib.amap_execute_static.argtypes = [c_void_p, POINTER(c_void_p), c_void_p, c_void_p]
    return lib


_lib = _load()
LIBRARY_PATH = _build.LIB


def _check(rc, where):
    if rc != 0:
        raise AmapError(rc, where)


def _i64(a):
    return (c_int64 * max(len(a), 1))(*[int(v) for v in a])


def _i32(a):
    return (c_int32 * max(len(a), 1))(*[int(v) for v in a])


class Builder:
    """amap_builder_*: emits the load/store statements of layout operators."""

    def __init__(self, elem_size: int):
        self._h = c_void_p()
        _check(_lib.amap_builder_create(c_int32(elem_size), byref(self._h)), "amap_builder_create")
        self.elem_size = elem_size

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:  # module globals are gone at interpreter shutdown
            _lib.amap_builder_destroy(self._h)
            self._h = None

    def _out(self, rc, where, out):
        _check(rc, where)
        return out.value

    def input(self, shape):
        o = c_int32()
        return self._out(_lib.amap_builder_input(self._h, len(shape), _i64(shape), byref(o)), "amap_builder_input", o)

    def tensor(self, shape):
        o = c_int32()
        return self._out(_lib.amap_builder_tensor(self._h, len(shape), _i64(shape), byref(o)), "amap_builder_tensor", o)

    def opaque(self, ins, shape):
        """The result of an operator that is not a layout operator, computed from tensors `ins`: bound at execute
        like an input."""
        o = c_int32()
        return self._out(
            _lib.amap_builder_opaque(self._h, len(ins), _i32(ins), len(shape), _i64(shape), byref(o)), "amap_builder_opaque", o
        )

    def reshape(self, src, shape):
        o = c_int32()
        return self._out(_lib.amap_builder_reshape(self._h, src, len(shape), _i64(shape), byref(o)), "amap_builder_reshape", o)

    def transpose(self, src, perm):
        o = c_int32()
        return self._out(_lib.amap_builder_transpose(self._h, src, len(perm), _i32(perm), byref(o)), "amap_builder_transpose", o)

    def slice(self, src, start, stop, step):
        o = c_int32()
        return self._out(
            _lib.amap_builder_slice(self._h, src, len(start), _i64(start), _i64(stop), _i64(step), byref(o)),
            "amap_builder_slice", o,
        )

    def concat(self, srcs, axis):
        o = c_int32()
        return self._out(_lib.amap_builder_concat(self._h, len(srcs), _i32(srcs), axis, byref(o)), "amap_builder_concat", o)

    def pad(self, src, lo, hi, fill_bits=0):
        o = c_int32()
        return self._out(
            _lib.amap_builder_pad(self._h, src, len(lo), _i64(lo), _i64(hi), c_uint64(fill_bits), byref(o)),
            "amap_builder_pad", o,
        )

    def window(self, src, kh, kw, stride, pad, dilation=1, order="rsc"):
        o = c_int32()
        if dilation == 1 and order == "rsc":
            return self._out(_lib.amap_builder_window(self._h, src, kh, kw, stride, pad, byref(o)), "amap_builder_window", o)
        return self._out(
            _lib.amap_builder_window_ex(self._h, src, kh, kw, stride, pad, dilation, {"rsc": 0, "crs": 1}[order], byref(o)),
            "amap_builder_window_ex", o,
        )

    def tile(self, src, reps):
        o = c_int32()
        return self._out(_lib.amap_builder_tile(self._h, src, len(reps), _i64(reps), byref(o)), "amap_builder_tile", o)

    def repeat(self, src, axis, count):
        out = c_int32()
        return self._out(_lib.amap_builder_repeat(self._h, src, int(axis), c_int64(int(count)), byref(out)), "amap_builder_repeat", out)

    def split(self, src, axis, sizes):
        """The ids of the parts, in order."""
        outs = (c_int32 * len(sizes))()
        _check(_lib.amap_builder_split(self._h, src, int(axis), len(sizes), _i64(sizes), outs), "amap_builder_split")
        return list(outs)

    def stmt(self, bounds, load, store, guarded=False, fill_bits=0):
        """One raw statement.  load = None | (tensor, C rows, b); store = (tensor, C rows, b)."""
        n = len(bounds)
        st = _Stmt()
        st.n_loops = n
        keep = [_i64(bounds)]
        st.bounds = keep[0]

        def acc(a):
            t, C, b = a
            flat = [v for row in C for v in row]
            Cb, bb = _i64(flat), _i64(b)
            keep.extend([Cb, bb])
            return _Access(int(t), len(b), Cb, bb)

        if load is None:
            st.load = _Access(AMAP_CONST, 0, None, None)
        else:
            st.load = acc(load)
        st.store = acc(store)
        st.guarded = int(bool(guarded))
        st.fill_bits = int(fill_bits)
        _check(_lib.amap_builder_stmt(self._h, byref(st)), "amap_builder_stmt")

    def compose(self, output, flags=0) -> "Map":
        chain = c_void_p()
        _check(_lib.amap_builder_chain(self._h, output, byref(chain)), "amap_builder_chain")
        h = c_void_p()
        if flags:
            _check(_lib.amap_compose_ex(chain, ctypes.c_uint32(flags), byref(h)), "amap_compose_ex")
        else:
            _check(_lib.amap_compose(chain, byref(h)), "amap_compose")
        return Map(h)

    def compose_multi(self, outputs, flags=0) -> "Map":
        """One map with several outputs (amap_compose_multi)."""
        chain = c_void_p()
        _check(_lib.amap_builder_chain(self._h, outputs[0] if outputs else 0, byref(chain)), "amap_builder_chain")
        h = c_void_p()
        _check(
            _lib.amap_compose_multi(chain, len(outputs), _i32(outputs), ctypes.c_uint32(flags), byref(h)), "amap_compose_multi"
        )
        return Map(h)


class Map:
    """A composed map: amap_compose's result."""

    def __init__(self, handle):
        self._h = handle
        n_in, out_numel, es = c_int32(), c_int64(), c_int32()
        _check(_lib.amap_map_sizes(self._h, byref(n_in), None, byref(out_numel), byref(es)), "amap_map_sizes")
        ins = (c_int64 * max(n_in.value, 1))()
        _check(_lib.amap_map_sizes(self._h, None, ins, None, None), "amap_map_sizes")
        self.in_numel = [ins[q] for q in range(n_in.value)]
        self.out_numel = out_numel.value
        self.elem_size = es.value
        n_out = c_int32()
        _check(_lib.amap_map_num_outputs(self._h, byref(n_out)), "amap_map_num_outputs")
        self.out_numels = []
        for k in range(n_out.value):
            n = c_int64()
            _check(_lib.amap_map_output_numel(self._h, k, byref(n)), "amap_map_output_numel")
            self.out_numels.append(n.value)

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:  # module globals are gone at interpreter shutdown
            _lib.amap_map_destroy(self._h)
            self._h = None

    def pieces(self):
        n = c_int32()
        _check(_lib.amap_map_num_pieces(self._h, byref(n)), "amap_map_num_pieces")
        out = []
        for k in range(n.value):
            p = _Piece()
            _check(_lib.amap_map_get_piece(self._h, k, byref(p)), "amap_map_get_piece")
            nl = p.n_loops

            def cons(ptr, cnt):
                return [([ptr[c].coef[j] for j in range(nl)], ptr[c].offset, ptr[c].extent) for c in range(cnt)]

            out.append(
                {
                    "bounds": [p.bounds[j] for j in range(nl)],
                    "input": p.input,
                    "C_l": [p.C_l[j] for j in range(nl)] if p.input >= 0 else None,
                    "b_l": p.b_l,
                    "C_s": [p.C_s[j] for j in range(nl)],
                    "b_s": p.b_s,
                    "guards": cons(p.guards, p.n_guards),
                    "domain": cons(p.domain, p.n_domain),
                    "fill_bits": p.fill_bits,
                    "output": p.output,
                    "quasi": None if p.n_digits == 0 else {
                        "radix": [p.digit_radix[d] for d in range(p.n_digits)],
                        "stride": [p.digit_stride[d] for d in range(p.n_digits)],
                        "F": [p.F[j] for j in range(nl)], "f0": p.f0,
                    },
                }
            )
        return out

    def stages(self):
        """[(first_piece, n_pieces, dst_temp (-1 = output), numel)] in execution order."""
        n = c_int32()
        _check(_lib.amap_map_num_stages(self._h, byref(n)), "amap_map_num_stages")
        out = []
        for s in range(n.value):
            fp, np_, dt, ne = c_int32(), c_int32(), c_int32(), c_int64()
            _check(_lib.amap_map_get_stage(self._h, s, byref(fp), byref(np_), byref(dt), byref(ne)), "amap_map_get_stage")
            out.append((fp.value, np_.value, dt.value, ne.value))
        return out

    def device_view(self) -> DeviceView:
        """amap_map_device_view: the map flattened for a consumer kernel that reads through it."""
        v = DeviceView()
        _check(_lib.amap_map_device_view(self._h, byref(v)), "amap_map_device_view")
        return v

    def rows_gather_host(self, inputs, cols):
        """amap_view_rows_gather_host: the result as rows of `cols` elements, gathered on the host through the row
        tables of the device view (numpy inputs; returns a flat numpy array of the inputs' dtype)."""
        import numpy as np

        v = self.device_view()
        xs = [np.ascontiguousarray(x) for x in inputs]
        arr = (c_void_p * max(len(xs), 1))(*[c_void_p(x.ctypes.data) for x in xs])
        out = np.empty(self.out_numel, dtype=xs[0].dtype)
        _check(_lib.amap_view_rows_gather_host(byref(v), c_int64(cols), arr, c_void_p(out.ctypes.data)), "amap_view_rows_gather_host")
        return out

    def consume_row_sums(self, srcs, rows, cols, sums, stream=None):
        """amap_consume_row_sums: uint32 sums of the rows of the chain's result, read through the map from the
        inputs (CUDA tensors `srcs`); `sums`: a CUDA int32/uint32 tensor of `rows` elements."""
        import torch

        v = self.device_view()
        arr = (c_void_p * max(len(srcs), 1))(*[c_void_p(t.data_ptr()) for t in srcs])
        s = (stream or torch.cuda.current_stream(sums.device)).cuda_stream
        _check(
            _lib.amap_consume_row_sums(byref(v), arr, c_int64(rows), c_int64(cols), c_void_p(sums.data_ptr()), c_void_p(s)),
            "amap_consume_row_sums",
        )

    def bind_consume_row_sums(self, srcs, rows, cols, sums, stream=None):
        """consume_row_sums with the arguments marshalled once; the returned callable only makes the C call."""
        import torch

        v = self.device_view()
        arr = (c_void_p * max(len(srcs), 1))(*[c_void_p(t.data_ptr()) for t in srcs])
        s = c_void_p((stream or torch.cuda.current_stream(sums.device)).cuda_stream)
        vp, r, c, d, fn = byref(v), c_int64(rows), c_int64(cols), c_void_p(sums.data_ptr()), _lib.amap_consume_row_sums

        def call():
            rc = fn(vp, arr, r, c, d, s)
            if rc != 0:
                raise AmapError(rc, "amap_consume_row_sums")

        call.keep = (v, list(srcs), sums, self)
        return call

    def plan(self, device=0, force_kernel=KERNEL_AUTO, pointer_align=16, flags=0) -> "Plan":
        opts = _PlanOpts()
        opts.force_kernel = force_kernel
        opts.pointer_align = pointer_align
        opts.flags = flags
        h = c_void_p()
        _check(_lib.amap_plan(self._h, device, byref(opts), byref(h)), "amap_plan")
        return Plan(h, self)


class Plan:
    """amap_plan's result; execute() enqueues the copy on a CUDA stream."""

    def __init__(self, handle, amap: Map):
        self._h = handle
        self.map = amap

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:  # module globals are gone at interpreter shutdown
            _lib.amap_plan_destroy(self._h)
            self._h = None

    def stats(self) -> dict:
        s = _Stats()
        _check(_lib.amap_plan_stats(self._h, byref(s)), "amap_plan_stats")
        return {
            "bytes_read": s.bytes_read, "bytes_written": s.bytes_written, "bytes_filled": s.bytes_filled,
            "n_pieces": s.n_pieces, "n_launches": s.n_launches, "n_stages": s.n_stages, "n_descriptors": s.n_descriptors,
            "kernels": {"gather": s.kernel_kind[0], "copy": s.kernel_kind[1], "transpose": s.kernel_kind[2], "fill": s.kernel_kind[3]},
        }

    def piece_kernels(self):
        out = []
        for k in range(self.stats()["n_pieces"]):
            kind = c_int32()
            _check(_lib.amap_plan_piece_kernel(self._h, k, byref(kind)), "amap_plan_piece_kernel")
            out.append(KERNEL_NAMES[kind.value])
        return out

    def launches(self):
        """One dict per kernel launch of an execute, in order: kernel name, access width, blocks, threads, ..."""
        out = []
        for k in range(self.stats()["n_launches"]):
            info = _LaunchInfo()
            _check(_lib.amap_plan_launch_info(self._h, k, byref(info)), "amap_plan_launch_info")
            d = {name: getattr(info, name) for name, _ in _LaunchInfo._fields_}
            d["kernel"] = LAUNCH_NAMES[info.kernel]
            out.append(d)
        return out

    def _src_array(self, src_ptrs):
        """n_inputs pointers; inputs left out at the end (not read by this map) are passed as NULL."""
        n = max(len(self.map.in_numel), len(src_ptrs), 1)
        ptrs = list(src_ptrs) + [None] * (n - len(src_ptrs))
        return (c_void_p * n)(*[c_void_p(p) for p in ptrs])

    def execute_ptrs(self, src_ptrs, dst_ptr, stream=0):
        arr = self._src_array(src_ptrs)
        _check(_lib.amap_execute(self._h, arr, c_void_p(dst_ptr), c_void_p(stream)), "amap_execute")

    def execute_multi_ptrs(self, src_ptrs, dst_ptrs, stream=0):
        """amap_execute_multi: one destination pointer per output of the map."""
        arr = self._src_array(src_ptrs)
        darr = (c_void_p * max(len(dst_ptrs), 1))(*[c_void_p(p) for p in dst_ptrs])
        _check(_lib.amap_execute_multi(self._h, arr, darr, c_void_p(stream)), "amap_execute_multi")

    def execute_static_ptrs(self, src_ptrs, dst_ptr, stream=0):
        """amap_execute_static: no device allocation; the descriptors go through the library's fixed table."""
        arr = self._src_array(src_ptrs)
        _check(_lib.amap_execute_static(self._h, arr, c_void_p(dst_ptr), c_void_p(stream)), "amap_execute_static")

    def bind(self, srcs, dst, stream=None):
        """Marshal the arguments of amap_execute once; the returned callable only makes the C call.
        Keeps `srcs` and `dst` alive.  For loops that launch the same plan on the same buffers many times."""
        import torch

        arr = self._src_array([t.data_ptr() for t in srcs])
        if isinstance(dst, (list, tuple)):  # a map with several outputs
            s = (stream or torch.cuda.current_stream(dst[0].device)).cuda_stream
            d = (c_void_p * len(dst))(*[c_void_p(t.data_ptr()) for t in dst])
            fn = _lib.amap_execute_multi
        else:
            s = (stream or torch.cuda.current_stream(dst.device)).cuda_stream
            d, fn = c_void_p(dst.data_ptr()), _lib.amap_execute
        h, st = self._h, c_void_p(s)
        keep = (list(srcs), dst, self)

        def call():
            rc = fn(h, arr, d, st)
            if rc != 0:
                raise AmapError(rc, "amap_execute")

        call.keep = keep
        return call

    def execute(self, srcs, dst, stream=None):
        """srcs: CUDA tensors (contiguous), dst: CUDA tensor; stream: torch.cuda.Stream or None (current)."""
        import torch

        for t in list(srcs) + [dst]:
            if not t.is_cuda or not t.is_contiguous():
                raise ValueError("amap_execute wants contiguous CUDA tensors")
        for t, n in zip(srcs, self.map.in_numel):
            if t.numel() * t.element_size() != n * self.map.elem_size:
                raise ValueError("input size differs from the composed map's")
        if dst.numel() * dst.element_size() != self.map.out_numel * self.map.elem_size:
            raise ValueError("output size differs from the composed map's")
        s = (stream or torch.cuda.current_stream(dst.device)).cuda_stream
        self.execute_ptrs([t.data_ptr() for t in srcs], dst.data_ptr(), s)

    def execute_host(self, srcs, dst, stream=0):
        """srcs / dst: host numpy arrays (or anything with .ctypes.data / .data_ptr())."""

        def ptr(a):
            return a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data

        arr = (c_void_p * max(len(srcs), 1))(*[c_void_p(ptr(a)) for a in srcs])
        _check(_lib.amap_execute_host(self._h, arr, c_void_p(ptr(dst)), c_void_p(stream)), "amap_execute_host")


def build_chain(chain) -> tuple:
    """Feed a workloads.Chain to the library's builder.  Returns (builder, output tensor id)."""
    b = Builder(chain.elem_size)
    ids = [b.input(s) for s in chain.inputs]
    for op in chain.ops:
        k = op["kind"]
        if k == "reshape":
            t = b.reshape(ids[op["src"]], op["shape"])
        elif k == "transpose":
            t = b.transpose(ids[op["src"]], op["perm"])
        elif k == "slice":
            t = b.slice(ids[op["src"]], op["start"], op["stop"], op["step"])
        elif k == "concat":
            t = b.concat([ids[s] for s in op["srcs"]], op["axis"])
        elif k == "pad":
            t = b.pad(ids[op["src"]], op["lo"], op["hi"], 0)
        elif k == "window":
            t = b.window(ids[op["src"]], op["kh"], op["kw"], op["stride"], op["pad"], op.get("dilation", 1), op.get("order", "rsc"))
        elif k == "tile":
            t = b.tile(ids[op["src"]], op["reps"])
        elif k == "repeat":
            t = b.repeat(ids[op["src"]], op["axis"], op["count"])
        elif k == "split":
            t = b.split(ids[op["src"]], op["axis"], op["sizes"])[op["part"]]
        elif k == "stmts":
            t = b.tensor(op["shape"])
            for st in op["stmts"]:
                load = None
                if st["load"] is not None:
                    lt, Cl, bl = st["load"]
                    load = (ids[lt], Cl, bl)
                Cs, bs = st["store"]
                b.stmt(st["bounds"], load, (t, Cs, bs), st.get("guarded", False), st.get("fill", 0))
        else:
            raise ValueError("unknown operator kind %r" % k)
        ids.append(t)
    b.ids = ids  # tensor id of every input and operator result, in the chain's numbering
    return b, ids[-1]


def compose_chain(chain, flags=0, outputs=None) -> Map:
    """`outputs`: tensor numbers of the chain (inputs first, then one per operator) wanted as results; default the
    last operator's."""
    b, out = build_chain(chain)
    if outputs is None:
        return b.compose(out, flags)
    return b.compose_multi([b.ids[t] for t in outputs], flags)
