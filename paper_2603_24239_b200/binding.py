"""ctypes binding of libdvm.so: argument marshalling only.

Every step of the hot path (shape tiling, bytecode encoding, the virtual
machine) runs inside the library.  If the library is missing the import fails
loudly -- there is no other implementation to fall back to.
"""
from __future__ import annotations

import ctypes as C

import numpy as np
import os
from typing import Iterable, List, Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libdvm.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is not built. Run `python -m paper_2603_24239_b200.build` "
        "(or __graft_entry__.build()); the library has no CPU fallback.")
lib = C.CDLL(LIB_PATH)

DVM_MAX_RANK = 6
F32, BF16, U8, I32 = 0, 1, 2, 3
DTYPES = {"f32": F32, "bf16": BF16, "u8": U8, "i32": I32}   # u8 / i32: outputs and casts (Table 1, Cast)
UNARY = {"exp": 0, "sqrt": 1, "rsqrt": 2, "abs": 3, "log": 4, "erf": 5, "sigmoid": 6, "neg": 7,
         "recip": 8, "floor": 9, "round": 10, "tanh": 11, "isfinite": 12}
BINARY = {"add": 0, "sub": 1, "mul": 2, "div": 3, "min": 4, "max": 5, "pow": 6}
SCALAR = {"adds": 0, "muls": 1}
REDUCE = {"sum": 0, "max": 1, "min": 2}
COMPARE = {"gt": 0, "ge": 1, "lt": 2, "le": 3, "eq": 4, "ne": 5}


class Shape(C.Structure):
    _fields_ = [("rank", C.c_int32), ("dims", C.c_int64 * DVM_MAX_RANK)]


class Strides(C.Structure):
    _fields_ = [("stride", C.c_int64 * DVM_MAX_RANK)]


class DvmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib.dvm_strerror(status).decode()
        if status == -6:
            msg += f" (cudaError {lib.dvm_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")


_vp, _i, _sz = C.c_void_p, C.c_int, C.c_size_t
_pi = C.POINTER(C.c_int)
_p64 = C.POINTER(C.c_int64)
_sig = {
    "dvm_program_create": ([C.POINTER(_vp)], _i),
    "dvm_program_destroy": ([_vp], None),
    "dvm_program_input": ([_vp, _i, _i, _pi], _i),
    "dvm_program_unary": ([_vp, _i, _i, _pi], _i),
    "dvm_program_binary": ([_vp, _i, _i, _i, _pi], _i),
    "dvm_program_scalar": ([_vp, _i, _i, C.c_float, _pi], _i),
    "dvm_program_scalar_param": ([_vp, _i, _i, _i, _pi], _i),
    "dvm_program_compare": ([_vp, _i, _i, _i, _pi], _i),
    "dvm_program_select": ([_vp, _i, _i, _i, _pi], _i),
    "dvm_program_cast": ([_vp, _i, _i, _pi], _i),
    "dvm_program_reduce": ([_vp, _i, _i, _i, _pi], _i),
    "dvm_program_matmul": ([_vp, _i, _i, _pi], _i),
    "dvm_program_output": ([_vp, _i, _i], _i),
    "dvm_program_finalize": ([_vp], _i),
    "dvm_program_num_inputs": ([_vp], _i),
    "dvm_program_num_outputs": ([_vp], _i),
    "dvm_encode": ([_vp, C.POINTER(Shape), _i, C.POINTER(C.c_float), _i, _vp, _sz, C.POINTER(_sz),
                    C.POINTER(Shape), _i], _i),
    "dvm_encode_strided": ([_vp, C.POINTER(Shape), C.POINTER(Strides), _i, C.POINTER(C.c_float), _i, C.POINTER(Strides),
                            _vp, _sz, C.POINTER(_sz), C.POINTER(Shape), _i], _i),
    "dvm_encode_batch": ([_i, C.POINTER(_vp), C.POINTER(Shape), _pi, C.POINTER(C.c_float), _pi, C.POINTER(_vp),
                          C.POINTER(_sz), C.POINTER(_sz), _pi], _i),
    "dvm_time_encode": ([_vp, C.POINTER(Shape), _vp, _i, C.POINTER(C.c_float), _i, _vp, _sz, _i, _p64], _i),
    "dvm_code_max_size": ([_vp], _sz),
    "dvm_set_num_cores": ([_i], None),
    "dvm_get_num_cores": ([], _i),
    "dvm_set_elems_per_thread": ([_i], None),
    "dvm_get_elems_per_thread": ([], _i),
    "dvm_set_min_resident_ctas": ([_i], None),
    "dvm_get_min_resident_ctas": ([], _i),
    "dvm_set_lean_kernel": ([_i], None),
    "dvm_last_launch_variant": ([C.POINTER(C.c_int)], _i),
    "dvm_set_stacked_one_slot": ([_i], None),
    "dvm_set_matmul_tail_split": ([_i], None),
    "dvm_set_matmul_cta_pairs": ([_i], None),
    "dvm_matmul_tail_plan": ([C.c_int64, _i, _i, _i, C.POINTER(C.c_int32)], _i),
    "dvm_hardware_align_div": ([C.c_int64, _i, C.c_int64, C.c_int64, C.c_int64, _p64, _p64, _p64, _p64], _i),
    "dvm_vm_tile_range": ([C.c_int64, _i, _i, _p64, _p64], _i),
    "dvm_launch": ([_vp, _sz, C.POINTER(_vp), _i, _vp], _i),
    "dvm_launch_stacked": ([_i, C.POINTER(_vp), C.POINTER(_sz), C.POINTER(C.POINTER(_vp)), _pi, _vp], _i),
    "dvm_launch_stacked_levels": ([_i, C.POINTER(_vp), C.POINTER(_sz), C.POINTER(C.POINTER(_vp)), _pi, _pi, _vp], _i),
    "dvm_launch_stacked_noalloc": ([_i, C.POINTER(_vp), C.POINTER(_sz), C.POINTER(C.POINTER(_vp)), _pi, _vp], _i),
    "dvm_run_host": ([_vp, _sz, C.POINTER(_vp), C.POINTER(_sz), _i, _vp, _sz, _vp], _i),
    "dvm_verify": ([_vp, _sz], _i),
    "dvm_disassemble": ([_vp, _sz, C.c_char_p, _sz], _i),
    "dvm_code_info": ([_vp, _sz, _pi, _p64, _pi, _pi, _pi, _pi], _i),
    "dvm_selftest_bounded_wait": ([_i, _vp], _i),
    "dvm_last_device_status": ([_vp, _pi], _i),
    "dvm_last_cuda_error": ([], _i),
    "dvm_launch_count": ([], C.c_int64),
    "dvm_strerror": ([_i], C.c_char_p),
}
_sig.update({
    "dvm_fuser_create": ([C.POINTER(_vp), _vp], _i),
    "dvm_fuser_destroy": ([_vp], None),
    "dvm_fuser_set_temporal_stacking": ([_vp, _i], _i),
    "dvm_fuser_tensor": ([_vp, _i, C.POINTER(Shape), _vp, _pi], _i),
    "dvm_fuser_unary": ([_vp, _i, _i, _i, _vp, C.POINTER(Shape), _pi], _i),
    "dvm_fuser_binary": ([_vp, _i, _i, _i, _i, _vp, C.POINTER(Shape), _pi], _i),
    "dvm_fuser_scalar": ([_vp, _i, _i, C.c_float, _i, _vp, C.POINTER(Shape), _pi], _i),
    "dvm_fuser_reduce": ([_vp, _i, _i, _i, _vp, C.POINTER(Shape), _pi], _i),
    "dvm_tensor_extents": ([_vp, C.c_size_t, C.POINTER(C.c_int64), _i], _i),
    "dvm_launch_checked": ([_vp, C.c_size_t, C.POINTER(_vp), C.POINTER(C.c_size_t), _i, _vp], _i),
    "dvm_fuser_reduce_axis": ([_vp, _i, _i, _i, _i, _vp, C.POINTER(Shape), _pi], _i),
    "dvm_fuser_compare": ([_vp, _i, _i, _i, _i, _vp, C.POINTER(Shape), _pi], _i),
    "dvm_fuser_select": ([_vp, _i, _i, _i, _i, _vp, C.POINTER(Shape), _pi], _i),
    "dvm_fuser_cast": ([_vp, _i, _i, _i, _vp, C.POINTER(Shape), _pi], _i),
    "dvm_fuser_matmul": ([_vp, _i, _i, _i, _vp, C.POINTER(Shape), _pi], _i),
    "dvm_fuser_release": ([_vp, _i], _i),
    "dvm_fuser_flush": ([_vp], _i),
    "dvm_fuser_pending": ([_vp, _pi, _pi], _i),
    "dvm_fuser_stats": ([_vp, _p64, _p64, _p64, _p64], _i),
})
for _name, (_args, _res) in _sig.items():
    _f = getattr(lib, _name)
    _f.argtypes = _args
    _f.restype = _res
EXPORTS = tuple(_sig)


def _check(st: int, where: str):
    if st != 0:
        raise DvmError(st, where)


class Program:
    """A shape-agnostic fused operator program (dvm_program)."""

    def __init__(self):
        self._h = _vp()
        _check(lib.dvm_program_create(C.byref(self._h)), "dvm_program_create")
        self._max_code = 0

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h and lib is not None:
            lib.dvm_program_destroy(h)

    def _node(self, fn, *args) -> int:
        out = C.c_int(-1)
        _check(fn(self._h, *args, C.byref(out)), fn.__name__)
        return out.value

    def input(self, dtype, rank):
        return self._node(lib.dvm_program_input, DTYPES.get(dtype, dtype), rank)

    def unary(self, op, x):
        return self._node(lib.dvm_program_unary, UNARY.get(op, op), x)

    def binary(self, op, x, y):
        return self._node(lib.dvm_program_binary, BINARY.get(op, op), x, y)

    def scalar(self, op, x, s):
        return self._node(lib.dvm_program_scalar, SCALAR.get(op, op), x, float(s))

    def scalar_param(self, op, x, k):
        return self._node(lib.dvm_program_scalar_param, SCALAR.get(op, op), x, int(k))

    def cast(self, x, dtype):
        return self._node(lib.dvm_program_cast, x, DTYPES.get(dtype, dtype))

    def reduce(self, op, x, axis=-1):
        return self._node(lib.dvm_program_reduce, REDUCE.get(op, op), x, axis)

    def matmul(self, a, b):
        return self._node(lib.dvm_program_matmul, a, b)

    def compare(self, op, x, y):
        return self._node(lib.dvm_program_compare, COMPARE.get(op, op), x, y)

    def select(self, cond, x, y):
        return self._node(lib.dvm_program_select, cond, x, y)

    def output(self, x, dtype):
        _check(lib.dvm_program_output(self._h, x, DTYPES.get(dtype, dtype)), "dvm_program_output")

    def finalize(self):
        _check(lib.dvm_program_finalize(self._h), "dvm_program_finalize")
        self._max_code = lib.dvm_code_max_size(self._h)
        return self

    @property
    def n_inputs(self):
        return lib.dvm_program_num_inputs(self._h)

    @property
    def n_outputs(self):
        return lib.dvm_program_num_outputs(self._h)


def program_from_nodes(nodes: Iterable[tuple]) -> Program:
    """Builds a Program from the plain-data node list of the workload module."""
    p = Program()
    ids = {}
    for i, n in enumerate(nodes):
        k = n[0]
        if k == "input":
            ids[i] = p.input(n[1], n[2])
        elif k == "unary":
            ids[i] = p.unary(n[1], ids[n[2]])
        elif k == "binary":
            ids[i] = p.binary(n[1], ids[n[2]], ids[n[3]])
        elif k == "scalar":
            if isinstance(n[3], tuple):
                ids[i] = p.scalar_param(n[1], ids[n[2]], n[3][1])
            else:
                ids[i] = p.scalar(n[1], ids[n[2]], n[3])
        elif k == "cast":
            ids[i] = p.cast(ids[n[1]], n[2])
        elif k == "reduce":
            ids[i] = p.reduce(n[1], ids[n[2]], n[3] if len(n) > 3 else -1)
        elif k == "matmul":
            ids[i] = p.matmul(ids[n[1]], ids[n[2]])
        elif k == "compare":
            ids[i] = p.compare(n[1], ids[n[2]], ids[n[3]])
        elif k == "select":
            ids[i] = p.select(ids[n[1]], ids[n[2]], ids[n[3]])
        elif k == "output":
            p.output(ids[n[1]], n[2])
        else:
            raise ValueError(f"unknown node kind {k}")
    return p.finalize()


class Code:
    """An encoded bytecode program in host memory plus the inferred output shapes."""
    __slots__ = ("buf", "size", "out_shapes")

    def __init__(self, buf, size, out_shapes):
        self.buf, self.size, self.out_shapes = buf, size, out_shapes

    def bytes(self) -> bytes:
        return bytes(self.buf)[: self.size]


class Encoder:
    """Reusable argument block for dvm_encode (no Python allocation per call)."""

    def __init__(self, program: Program):
        self.program = program
        self.n_in, self.n_out = program.n_inputs, program.n_outputs
        self.shapes = (Shape * self.n_in)()
        self.out_shapes = (Shape * max(self.n_out, 1))()
        self.cap = program._max_code
        self.buf = (C.c_uint64 * ((self.cap + 7) // 8))()
        self.size = _sz(0)
        self.scalars = (C.c_float * 16)()

    def time_encode(self, shapes: Sequence[Sequence[int]], scalars: Sequence[float] = (), reps: int = 1000,
                    in_strides: Optional[Sequence[Optional[Sequence[int]]]] = None) -> List[int]:
        """Durations (ns, steady clock read inside the library) of `reps` encodes of one instance: the encoder
        alone, without the binding."""
        for s, shp in zip(self.shapes, shapes):
            s.rank = len(shp)
            for k, d in enumerate(shp):
                s.dims[k] = d
        for k, v in enumerate(scalars):
            self.scalars[k] = v
        ins = None
        if in_strides is not None:
            ins = (Strides * self.n_in)()
            for a, t, shp in zip(ins, in_strides, shapes):
                for k, v in enumerate(t if t is not None else _dense_strides(shp)):
                    a.stride[k] = v
        out = (C.c_int64 * reps)()
        st = lib.dvm_time_encode(self.program._h, self.shapes, ins, self.n_in, self.scalars, len(scalars),
                                 self.buf, self.cap, reps, out)
        if st != 0:
            raise DvmError(st, "dvm_time_encode")
        return list(out)

    def encode(self, shapes: Sequence[Sequence[int]], scalars: Sequence[float] = (),
               in_strides: Optional[Sequence[Optional[Sequence[int]]]] = None,
               out_strides: Optional[Sequence[Optional[Sequence[int]]]] = None) -> int:
        """in_strides / out_strides (element strides per dim, None = dense) select dvm_encode_strided."""
        for s, shp in zip(self.shapes, shapes):
            s.rank = len(shp)
            for k, d in enumerate(shp):
                s.dims[k] = d
        for k, v in enumerate(scalars):
            self.scalars[k] = v
        if in_strides is None and out_strides is None:
            st = lib.dvm_encode(self.program._h, self.shapes, self.n_in, self.scalars, len(scalars),
                                self.buf, self.cap, C.byref(self.size), self.out_shapes, self.n_out)
            if st != 0:
                raise DvmError(st, "dvm_encode")
            return self.size.value
        if out_strides is not None and any(t is None for t in out_strides):
            # a dense output among views: its strides follow from the output shape, which a plain encode reports
            st = lib.dvm_encode(self.program._h, self.shapes, self.n_in, self.scalars, len(scalars),
                                self.buf, self.cap, C.byref(self.size), self.out_shapes, self.n_out)
            if st != 0:
                raise DvmError(st, "dvm_encode")
            out_strides = [t if t is not None else _dense_strides(shp) for t, shp in zip(out_strides, self.output_shapes())]
        ins = None
        if in_strides is not None:
            ins = (Strides * self.n_in)()
            for a, t, shp in zip(ins, in_strides, shapes):
                for k, v in enumerate(t if t is not None else _dense_strides(shp)):
                    a.stride[k] = v
        outs = None
        if out_strides is not None:
            outs = (Strides * max(self.n_out, 1))()
            for a, t in zip(outs, out_strides):
                for k, v in enumerate(t):
                    a.stride[k] = v
        st = lib.dvm_encode_strided(self.program._h, self.shapes, ins, self.n_in, self.scalars, len(scalars), outs,
                                    self.buf, self.cap, C.byref(self.size), self.out_shapes, self.n_out)
        if st != 0:
            raise DvmError(st, "dvm_encode_strided")
        return self.size.value

    def output_shapes(self) -> List[tuple]:
        return [tuple(self.out_shapes[o].dims[k] for k in range(self.out_shapes[o].rank))
                for o in range(self.n_out)]


class BatchEncoder:
    """Reusable argument block for dvm_encode_batch: the instances of one stacked launch, encoded in one call.

    `programs` fixes the program of every instance; encode() takes this launch's shapes and scalars.
    The code buffers stay valid until the next encode(); launch_args() hands them to dvm_launch_stacked."""

    def __init__(self, programs: Sequence[Program]):
        n = self.n = len(programs)
        self.programs = list(programs)
        self.handles = (_vp * n)(*[p._h for p in programs])
        self.n_in = (_i * n)(*[p.n_inputs for p in programs])
        self.total_in = sum(p.n_inputs for p in programs)
        self.shapes = (Shape * self.total_in)()
        # the same memory as a numpy record array: one vectorised copy marshals every shape of the launch
        self._np_shapes = np.frombuffer(self.shapes, dtype=np.dtype({"names": ["rank", "dims"],
                                                                      "formats": ["<i4", ("<i8", DVM_MAX_RANK)],
                                                                      "offsets": [0, 8], "itemsize": C.sizeof(Shape)}))
        self.n_scalars = (_i * n)()
        self.scalars = (C.c_float * (16 * n))()
        caps = [p._max_code for p in programs]
        self.bufs = [(C.c_uint64 * ((c + 7) // 8))() for c in caps]
        self.codes = (_vp * n)(*[C.addressof(b) for b in self.bufs])
        self.caps = (_sz * n)(*caps)
        self.sizes = (_sz * n)()
        self.failed = _i(0)

    def encode(self, shapes: Sequence[Sequence[Sequence[int]]], scalars: Sequence[Sequence[float]]):
        """shapes[i]: the input shapes of instance i; scalars[i]: its runtime scalar arguments."""
        flat = [s for inst in shapes for s in inst]
        ranks = np.fromiter((len(s) for s in flat), dtype=np.int32, count=self.total_in)
        dims = np.zeros((self.total_in, DVM_MAX_RANK), dtype=np.int64)
        for k, s in enumerate(flat):
            dims[k, :len(s)] = s
        self._np_shapes["rank"] = ranks
        self._np_shapes["dims"] = dims
        k = 0
        for i, sc in enumerate(scalars):
            self.n_scalars[i] = len(sc)
            for v in sc:
                self.scalars[k] = v
                k += 1
        st = lib.dvm_encode_batch(self.n, self.handles, self.shapes, self.n_in, self.scalars, self.n_scalars,
                                  self.codes, self.caps, self.sizes, C.byref(self.failed))
        if st != 0:
            raise DvmError(st, f"dvm_encode_batch (instance {self.failed.value})")


def _dense_strides(shape: Sequence[int]) -> List[int]:
    out, st = [], 1
    for d in reversed(list(shape)):
        out.append(st)
        st *= max(int(d), 1)
    return out[::-1]


def encode(program: Program, shapes: Sequence[Sequence[int]], scalars: Sequence[float] = (),
           in_strides=None, out_strides=None) -> Code:
    """dvm_encode: one dynamic-shape instance -> bytecode.  With in_strides / out_strides (element strides per
    dim of each input / output view; None entries are dense): dvm_encode_strided."""
    enc = Encoder(program)
    size = enc.encode(shapes, scalars, in_strides, out_strides)
    return Code(enc.buf, size, enc.output_shapes())


def _ptr(t) -> int:
    return t if isinstance(t, int) else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return None
    return stream if isinstance(stream, int) else stream.cuda_stream


def launch(code: Code, tensors: Sequence, stream=None):
    """dvm_launch: tensors are device tensors (or raw device addresses), inputs then outputs."""
    arr = (_vp * len(tensors))(*[_ptr(t) for t in tensors])
    _check(lib.dvm_launch(code.buf, code.size, arr, len(tensors), _stream(stream)), "dvm_launch")


def tensor_extents(code: Code) -> List[int]:
    """dvm_tensor_extents: bytes of every tensor slot (inputs, then outputs) a launch of `code` addresses."""
    n = 0
    out = (C.c_int64 * 16)()
    for n in range(17):   # the slot count is part of the code: ask until it matches
        st = lib.dvm_tensor_extents(code.buf, code.size, out, n)
        if st == 0:
            return [int(out[i]) for i in range(n)]
        if st != -1:
            _check(st, "dvm_tensor_extents")
    raise DvmError(-1, "dvm_tensor_extents")


def launch_checked(code: Code, tensors: Sequence, tensor_bytes: Sequence[int], stream=None):
    """dvm_launch_checked: dvm_launch behind a bounds check of every tensor against the bytes the program addresses."""
    arr = (_vp * len(tensors))(*[_ptr(t) for t in tensors])
    sizes = (C.c_size_t * len(tensor_bytes))(*[int(b) for b in tensor_bytes])
    _check(lib.dvm_launch_checked(code.buf, code.size, arr, sizes, len(tensors), _stream(stream)), "dvm_launch_checked")


def launch_stacked(codes: Sequence[Code], tensor_lists: Sequence[Sequence], stream=None, noalloc: bool = False,
                   levels: Optional[Sequence[int]] = None):
    """dvm_launch_stacked: many independent programs in one kernel launch.

    levels (non-decreasing, one per program) calls dvm_launch_stacked_levels instead: a program may read what
    programs of lower levels of the same launch write.

    noalloc=True calls dvm_launch_stacked_noalloc, the variant for callers that may not allocate device
    memory (its work queue lives in a fixed array inside the library instead of a cudaMalloc'd buffer)."""
    n = len(codes)
    cptr = (_vp * n)(*[C.addressof(c.buf) for c in codes])
    csz = (_sz * n)(*[c.size for c in codes])
    keep = [(_vp * len(tl))(*[_ptr(t) for t in tl]) for tl in tensor_lists]
    tptr = (C.POINTER(_vp) * n)(*[C.cast(k, C.POINTER(_vp)) for k in keep])
    nt = (_i * n)(*[len(tl) for tl in tensor_lists])
    if levels is not None:
        lv = (_i * n)(*[int(v) for v in levels])
        _check(lib.dvm_launch_stacked_levels(n, cptr, csz, tptr, nt, lv, _stream(stream)), "dvm_launch_stacked_levels")
        return
    fn = lib.dvm_launch_stacked_noalloc if noalloc else lib.dvm_launch_stacked
    _check(fn(n, cptr, csz, tptr, nt, _stream(stream)), fn.__name__)


def run_host(code: Code, host_tensors: Sequence, staging, stream=None):
    """dvm_run_host: host tensors in, host tensors out; copies are inside the call."""
    n = len(host_tensors)
    arr = (_vp * n)(*[_ptr(t) for t in host_tensors])
    nbytes = (_sz * n)(*[t.numel() * t.element_size() for t in host_tensors])
    _check(lib.dvm_run_host(code.buf, code.size, arr, nbytes, n, _ptr(staging),
                            staging.numel() * staging.element_size(), _stream(stream)), "dvm_run_host")


def verify(code) -> int:
    if isinstance(code, Code):
        return lib.dvm_verify(code.buf, code.size)
    raw = bytes(code)
    buf = (C.c_uint64 * ((len(raw) + 7) // 8 + 1))()
    C.memmove(buf, raw, len(raw))
    return lib.dvm_verify(buf, len(raw))


def disassemble(code: Code) -> str:
    out = C.create_string_buffer(1 << 16)
    _check(lib.dvm_disassemble(code.buf, code.size, out, len(out)), "dvm_disassemble")
    return out.value.decode()


def code_info(code: Code) -> dict:
    kt, bb, tpr, vw, nr = C.c_int(), C.c_int(), C.c_int(), C.c_int(), C.c_int()
    nt = C.c_int64()
    _check(lib.dvm_code_info(code.buf, code.size, C.byref(kt), C.byref(nt), C.byref(bb), C.byref(tpr),
                             C.byref(vw), C.byref(nr)), "dvm_code_info")
    return {"kernel_type": kt.value, "n_tiles": nt.value, "code_body_bytes": bb.value,
            "threads_per_row": tpr.value, "vector_width": vw.value, "n_tile_regs": nr.value}


def last_device_status(stream=None) -> int:
    st = C.c_int(0)
    _check(lib.dvm_last_device_status(_stream(stream), C.byref(st)), "dvm_last_device_status")
    return st.value


class Fuser:
    """The streaming runtime operator fuser (dvm_fuser_*): operators arrive one at a time on device tensors,
    are fused as they arrive and run at flush().  `alloc(shape, dtype)` returns the device tensor for a result
    (default: torch.empty on cuda); pass alloc=None ... address pairs for CPU-only planning tests."""

    def __init__(self, stream=None, alloc=None, temporal_stacking: bool = True):
        self._h = _vp()
        _check(lib.dvm_fuser_create(C.byref(self._h), _stream(stream)), "dvm_fuser_create")
        _check(lib.dvm_fuser_set_temporal_stacking(self._h, int(temporal_stacking)), "dvm_fuser_set_temporal_stacking")
        self._alloc = alloc
        self.tensors = {}   # value id -> tensor (keeps result buffers alive)

    def __del__(self):
        if getattr(self, "_h", None):
            lib.dvm_fuser_destroy(self._h)
            self._h = None

    def tensor(self, t, dtype=None, shape=None) -> int:
        """A tensor already in device memory; t is a torch tensor, or a raw address with dtype and shape."""
        if isinstance(t, int):
            addr, dt, shp = t, DTYPES[dtype], tuple(shape)
        else:
            import torch
            addr, dt, shp = t.data_ptr(), (DTYPES["bf16"] if t.dtype == torch.bfloat16 else DTYPES["f32"]), tuple(t.shape)
        s = Shape()
        s.rank = len(shp)
        for k, d in enumerate(shp):
            s.dims[k] = d
        out = C.c_int(-1)
        _check(lib.dvm_fuser_tensor(self._h, dt, C.byref(s), addr, C.byref(out)), "dvm_fuser_tensor")
        self.tensors[out.value] = t
        return out.value

    def _result(self, shape_guess, dtype):
        import torch
        if self._alloc is not None:
            return self._alloc(shape_guess, dtype)
        tdt = {"bf16": torch.bfloat16, "f32": torch.float32, "u8": torch.uint8, "i32": torch.int32}[dtype]
        return torch.empty(shape_guess, dtype=tdt, device="cuda")

    def _op(self, fn, args, out_shape, dtype):
        buf = self._result(out_shape, dtype)
        addr = buf if isinstance(buf, int) else buf.data_ptr()
        s, out = Shape(), C.c_int(-1)
        _check(fn(self._h, *args, DTYPES[dtype], addr, C.byref(s), C.byref(out)), fn.__name__)
        got = tuple(s.dims[k] for k in range(s.rank))
        assert tuple(out_shape) == got, (out_shape, got)
        self.tensors[out.value] = buf
        return out.value

    def unary(self, op, x, out_shape, dtype="f32"):
        return self._op(lib.dvm_fuser_unary, (UNARY.get(op, op), x), out_shape, dtype)

    def binary(self, op, x, y, out_shape, dtype="f32"):
        return self._op(lib.dvm_fuser_binary, (BINARY.get(op, op), x, y), out_shape, dtype)

    def scalar(self, op, x, s, out_shape, dtype="f32"):
        return self._op(lib.dvm_fuser_scalar, (SCALAR.get(op, op), x, float(s)), out_shape, dtype)

    def reduce(self, op, x, out_shape, dtype="f32", axis=-1):
        if axis != -1:
            return self._op(lib.dvm_fuser_reduce_axis, (REDUCE.get(op, op), x, axis), out_shape, dtype)
        return self._op(lib.dvm_fuser_reduce, (REDUCE.get(op, op), x), out_shape, dtype)

    def compare(self, op, x, y, out_shape, dtype="f32"):
        return self._op(lib.dvm_fuser_compare, (COMPARE.get(op, op), x, y), out_shape, dtype)

    def select(self, cond, x, y, out_shape, dtype="f32"):
        return self._op(lib.dvm_fuser_select, (cond, x, y), out_shape, dtype)

    def cast(self, x, to, out_shape, dtype=None):
        """x rounded to type `to`; stored as `dtype` (default: `to`)."""
        return self._op(lib.dvm_fuser_cast, (x, DTYPES[to]), out_shape, dtype or to)

    def matmul(self, a, b, out_shape, dtype="bf16"):
        return self._op(lib.dvm_fuser_matmul, (a, b), out_shape, dtype)

    def release(self, value):
        _check(lib.dvm_fuser_release(self._h, value), "dvm_fuser_release")

    def flush(self):
        _check(lib.dvm_fuser_flush(self._h), "dvm_fuser_flush")

    def pending(self):
        a, b = C.c_int(0), C.c_int(0)
        _check(lib.dvm_fuser_pending(self._h, C.byref(a), C.byref(b)), "dvm_fuser_pending")
        return a.value, b.value

    def stats(self):
        v = [C.c_int64(0) for _ in range(4)]
        _check(lib.dvm_fuser_stats(self._h, *[C.byref(x) for x in v]), "dvm_fuser_stats")
        return dict(zip(("ops", "groups", "launches", "stores_elided"), (x.value for x in v)))


def selftest_bounded_wait(which: int, stream=None):
    """Launches the kernel whose wait must run out (about 2 s); read the outcome with last_device_status()."""
    _check(lib.dvm_selftest_bounded_wait(which, _stream(stream)), "dvm_selftest_bounded_wait")


def launch_count() -> int:
    return lib.dvm_launch_count()


def hardware_align_div(total, n_cores, align, t_max, overhead=2):
    a, b, c, d = C.c_int64(), C.c_int64(), C.c_int64(), C.c_int64()
    _check(lib.dvm_hardware_align_div(total, n_cores, align, t_max, overhead, C.byref(a), C.byref(b),
                                      C.byref(c), C.byref(d)), "dvm_hardware_align_div")
    return {"min_cost_tile": a.value, "rounded_tile": b.value, "n_tiles": c.value, "tail": d.value}


def vm_tile_range(n_tiles, n_cores, core_id):
    b, e = C.c_int64(), C.c_int64()
    _check(lib.dvm_vm_tile_range(n_tiles, n_cores, core_id, C.byref(b), C.byref(e)), "dvm_vm_tile_range")
    return b.value, e.value


def set_num_cores(n: int):
    lib.dvm_set_num_cores(n)


def get_num_cores() -> int:
    return lib.dvm_get_num_cores()


def set_elems_per_thread(v: int):
    lib.dvm_set_elems_per_thread(v)


def set_lean_kernel(on: bool):
    """False: every launch runs on the general interpreter (for comparisons); True (default): programs of the
    basic instruction set run on the lean variant."""
    lib.dvm_set_lean_kernel(int(on))


def set_matmul_tail_split(on: bool):
    """dvm_set_matmul_tail_split: split the tiles of a matmul launch's last, partial wave along k (default on)."""
    lib.dvm_set_matmul_tail_split(int(bool(on)))


def matmul_tail_plan(tiles: int, units: int, k_blocks: int, ctas_per_unit: int = 1):
    """dvm_matmul_tail_plan: None when such a launch does not split its last wave, else a dict of the plan."""
    out = (C.c_int32 * 6)()
    st = lib.dvm_matmul_tail_plan(tiles, units, k_blocks, ctas_per_unit, out)
    if st < 0:
        _check(st, "dvm_matmul_tail_plan")
    if st == 0:
        return None
    return {"first": out[0], "r": out[1], "parts_max": out[2], "kb_per_unit": out[3], "tile_pitch": out[4], "units_used": out[5]}


def last_launch_variant() -> dict:
    """dvm_last_launch_variant: the interpreter build the last vector launch of this thread ran on."""
    out = (C.c_int * 8)()
    _check(lib.dvm_last_launch_variant(out), "dvm_last_launch_variant")
    return dict(zip(("V", "large", "single", "ext", "levels", "lean", "heavy", "ctas"), list(out)))


def set_matmul_cta_pairs(mode: int):
    """dvm_set_matmul_cta_pairs: matmul launches on CTA pairs (0 never, 1 default: by shape, 2 wherever possible)."""
    lib.dvm_set_matmul_cta_pairs(int(mode))


def set_stacked_one_slot(on: bool):
    """dvm_set_stacked_one_slot: stacked launches run with one tile slot per CTA (programs encoded with
    set_min_resident_ctas(3))."""
    lib.dvm_set_stacked_one_slot(int(bool(on)))


def set_min_resident_ctas(n: int):
    """2: encode only geometries whose tile slots fit twice per SM (programs of a stacked launch); 0: no constraint."""
    lib.dvm_set_min_resident_ctas(n)
