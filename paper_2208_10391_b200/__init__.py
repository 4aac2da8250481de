"""Python binding of the C-ABI library declared in ``include/mom.h``.

Argument marshalling only: every function here forwards to the `extern "C"` entry point of the same
name in ``libmom.so``; planning runs in the library's C++ planner and every product in its CUDA
kernels.  There is no Python or CPU fallback: if the shared library is missing, importing this
package raises.  Device pointers are plain integers (e.g. ``tensor.data_ptr()``); streams are
integer handles (e.g. ``torch.cuda.current_stream().cuda_stream``).
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

GENERAL, LOWER_TRI, UPPER_TRI, IDENTITY, DIAGONAL, SYMMETRIC = 0, 1, 2, 3, 4, 5
STRICT_LOWER, STRICT_UPPER, UNIT_LOWER, UNIT_UPPER = 6, 7, 8, 9
F32 = 0
VARIANT_3XTF32, VARIANT_FFMA, VARIANT_3XTF32_FORCE, VARIANT_3XTF32_WARP, VARIANT_3XTF32_INLINE = 0, 1, 2, 3, 4
STORAGE_DENSE, STORAGE_PACKED = 0, 1
KIND_GG, KIND_TG, KIND_GT, KIND_TT, KIND_TTMIX, KIND_SCALE, KIND_GRAM = 0, 1, 2, 3, 4, 5, 6

(OK, ERR_INVALID_ARG, ERR_PROPERTY, ERR_DTYPE, ERR_SHAPE_MISMATCH, ERR_OVERFLOW, ERR_ALLOC,
 ERR_WORKSPACE_TOO_SMALL, ERR_ALIGNMENT, ERR_ARCH, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_BUFFER_TOO_SMALL,
 ERR_LIMIT) = range(14)

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmom.so")


class MatrixDesc(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int64), ("cols", ctypes.c_int64),
                ("property", ctypes.c_int32), ("dtype", ctypes.c_int32)]


class Step(ctypes.Structure):
    _fields_ = [("lhs", ctypes.c_int32), ("rhs", ctypes.c_int32), ("out", ctypes.c_int32),
                ("kind", ctypes.c_int32), ("lhs_property", ctypes.c_int32), ("rhs_property", ctypes.c_int32),
                ("out_property", ctypes.c_int32), ("uses_tensor_cores", ctypes.c_int32),
                ("lhs_transposed", ctypes.c_int32), ("rhs_transposed", ctypes.c_int32),
                ("m", ctypes.c_int64), ("n", ctypes.c_int64), ("k", ctypes.c_int64),
                ("useful_mults", ctypes.c_uint64)]


class ExprNode(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("operand", ctypes.c_int32), ("first_child", ctypes.c_int32),
                ("n_children", ctypes.c_int32)]


class MomError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {status_string(status)} (status {int(status)})")


if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python paper_2208_10391_b200/csrc/build.py` "
        "(there is no fallback implementation)")

_lib = ctypes.CDLL(LIB_PATH)

_P = ctypes.c_void_p
_sigs = {
    "mom_matrix_desc": [ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.POINTER(MatrixDesc)],
    "mom_column_slab": [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int64, ctypes.POINTER(ctypes.c_int64),
                        ctypes.POINTER(ctypes.c_int64)],
    "mom_column_slab_desc": [ctypes.POINTER(MatrixDesc), ctypes.c_int32, ctypes.c_int64, ctypes.c_int64,
                             ctypes.POINTER(MatrixDesc)],
    "mom_equation_plan": [ctypes.POINTER(MatrixDesc), ctypes.c_int32, ctypes.POINTER(MatrixDesc), ctypes.c_int32,
                          ctypes.c_int, ctypes.POINTER(_P)],
    "mom_equation_plan_transposed": [ctypes.POINTER(MatrixDesc), ctypes.POINTER(ctypes.c_int32), ctypes.c_int32,
                                     ctypes.POINTER(MatrixDesc), ctypes.POINTER(ctypes.c_int32), ctypes.c_int32,
                                     ctypes.c_int, ctypes.POINTER(_P)],
    "mom_packed_elements": [ctypes.c_int64, ctypes.c_int, ctypes.POINTER(ctypes.c_int64)],
    "mom_packed_row": [ctypes.c_int64, ctypes.c_int, ctypes.c_int64, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
                       ctypes.POINTER(ctypes.c_int64)],
    "mom_equation_plan_stored": [ctypes.POINTER(MatrixDesc), ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32), ctypes.c_int32,
                                 ctypes.POINTER(MatrixDesc), ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32), ctypes.c_int32,
                                 ctypes.c_int, ctypes.c_int, ctypes.POINTER(_P)],
    "mom_plan_result_elements": [_P, ctypes.POINTER(ctypes.c_int64)],
    "mom_equation_plan_sum": [ctypes.POINTER(MatrixDesc), ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32),
                              ctypes.POINTER(ctypes.c_int32), ctypes.c_int32, ctypes.c_int, ctypes.POINTER(_P)],
    "mom_plan_reused_products": [_P, ctypes.POINTER(ctypes.c_int32)],
    "mom_expression_plan": [ctypes.POINTER(MatrixDesc), ctypes.c_int32, ctypes.POINTER(ExprNode), ctypes.c_int32,
                            ctypes.POINTER(ctypes.c_int32), ctypes.c_int32, ctypes.c_int32, ctypes.c_int,
                            ctypes.POINTER(_P)],
    "mom_plan_temporaries": [_P, ctypes.POINTER(ctypes.c_int32)],
    "mom_plan_flops": [_P, ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64)],
    "mom_plan_parenthesization": [_P, ctypes.c_char_p, ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)],
    "mom_plan_num_steps": [_P, ctypes.POINTER(ctypes.c_int32)],
    "mom_plan_step": [_P, ctypes.c_int32, ctypes.POINTER(Step)],
    "mom_plan_result_desc": [_P, ctypes.POINTER(MatrixDesc)],
    "mom_plan_workspace_bytes": [_P, ctypes.c_int64, ctypes.POINTER(ctypes.c_size_t)],
    "mom_equation_execute": [_P, ctypes.POINTER(_P), ctypes.POINTER(_P), _P, _P, ctypes.c_size_t, _P],
    "mom_equation_execute_batched": [_P, ctypes.POINTER(_P), ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(_P),
                                     ctypes.POINTER(ctypes.c_int64), _P, ctypes.c_int64, ctypes.c_int64, _P,
                                     ctypes.c_size_t, _P],
    "mom_plan_host_staging_bytes": [_P, ctypes.c_int64, ctypes.POINTER(ctypes.c_size_t)],
    "mom_plan_host_upload_bytes": [_P, ctypes.c_int64, ctypes.POINTER(ctypes.c_size_t)],
    "mom_equation_execute_host": [_P, ctypes.POINTER(_P), ctypes.POINTER(_P), _P, ctypes.c_int64, _P,
                                  ctypes.c_size_t, _P],
    "mom_plan_device_status": [_P, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)],
    "mom_probe_wait_timeout": [_P, ctypes.c_double, ctypes.c_int32, _P],
    "mom_plan_concurrent_steps": [_P, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)],
    "mom_plan_last_launch_count": [_P, ctypes.POINTER(ctypes.c_int32)],
    "mom_plan_enable_step_timing": [_P, ctypes.c_int32],
    "mom_plan_step_times": [_P, ctypes.c_int32, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float)],
    "mom_plan_destroy": [_P],
    "mom_product_3xtf32_noalloc": [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int, _P, _P, _P,
                                   _P, _P],
    "mom_probe_tf32_tflops": [ctypes.c_double, _P, _P, ctypes.POINTER(ctypes.c_double)],
    "mom_probe_ffma_tflops": [ctypes.c_double, _P, _P, ctypes.POINTER(ctypes.c_double)],
}
for _name, _args in _sigs.items():
    _fn = getattr(_lib, _name)
    _fn.argtypes = _args
    _fn.restype = ctypes.c_int
_lib.mom_status_string.argtypes = [ctypes.c_int]
_lib.mom_status_string.restype = ctypes.c_char_p

EXPORTED = sorted(list(_sigs) + ["mom_status_string"])


def status_string(status: int) -> str:
    return _lib.mom_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise MomError(status, where)


def _ptr_array(values: Sequence[Optional[int]]):
    arr = (_P * max(len(values), 1))()
    for i, v in enumerate(values):
        arr[i] = None if v is None else int(v)
    return arr


def mom_matrix_desc(rows: int, cols: int, prop: int = GENERAL, dtype: int = F32) -> MatrixDesc:
    d = MatrixDesc()
    _check(_lib.mom_matrix_desc(rows, cols, prop, dtype, ctypes.byref(d)), "mom_matrix_desc")
    return d


def _as_desc(d) -> MatrixDesc:
    if isinstance(d, MatrixDesc):
        return d
    return MatrixDesc(int(d[0]), int(d[1]), int(d[2]), F32 if len(d) < 4 else int(d[3]))


def mom_column_slab(cols: int, rank: int, world: int, multiple: int = 4) -> Tuple[int, int]:
    """Columns [begin, end) of X that device `rank` of `world` evaluates (begin == end: nothing to do)."""
    b, e = ctypes.c_int64(), ctypes.c_int64()
    _check(_lib.mom_column_slab(cols, rank, world, multiple, ctypes.byref(b), ctypes.byref(e)), "mom_column_slab")
    return b.value, e.value


def mom_column_slab_desc(stored, transposed: bool, begin: int, end: int) -> MatrixDesc:
    """Descriptor of the stored matrix that holds columns [begin, end) of an operand as used."""
    src, out = _as_desc(stored), MatrixDesc()
    _check(_lib.mom_column_slab_desc(ctypes.byref(src), 1 if transposed else 0, begin, end, ctypes.byref(out)),
           "mom_column_slab_desc")
    return out


def column_slab_equation(chain: Sequence, add_terms: Sequence, rank: int, world: int, chain_transposed: Sequence = (),
                         add_transposed: Sequence = (), multiple: int = 4):
    """Descriptors of device `rank`'s slab equation: the chain with its last operand cut to the slab's columns and
    every Add term likewise.  Returns (chain, add_terms, begin, end), or None when the slab is empty.  Marshalling
    only: the bounds and the slab descriptors come from the library."""
    chain = [_as_desc(d) for d in chain]
    add_terms = [_as_desc(d) for d in add_terms]
    ct = list(chain_transposed) + [False] * (len(chain) - len(chain_transposed))
    at = list(add_transposed) + [False] * (len(add_terms) - len(add_transposed))
    cols = chain[-1].rows if ct[-1] else chain[-1].cols
    begin, end = mom_column_slab(cols, rank, world, multiple)
    if begin == end:
        return None
    chain[-1] = mom_column_slab_desc(chain[-1], ct[-1], begin, end)
    add_terms = [mom_column_slab_desc(d, t, begin, end) for d, t in zip(add_terms, at)]
    return chain, add_terms, begin, end


def gather_column_slabs(x_slab, rows: int, cols: int, rank: int, world: int, multiple: int = 4, group=None):
    """All-gather of the devices' slabs of X into the whole rows x cols matrix on every rank (torch.distributed;
    NCCL on GPUs).  `x_slab` is this rank's rows x (end - begin) tensor (rows x 0 for an empty slab: it still
    supplies device and dtype).  The slabs are padded to the widest one for the collective; no arithmetic happens
    here."""
    import torch
    import torch.distributed as dist
    bounds = [mom_column_slab(cols, r, world, multiple) for r in range(world)]
    b, e = bounds[rank]
    if tuple(x_slab.shape) != (rows, e - b):
        raise ValueError(f"rank {rank} holds columns {b}..{e} of {rows} x {cols}, not a tensor of shape {tuple(x_slab.shape)}")
    width = max(hi - lo for lo, hi in bounds)
    buf = torch.zeros((rows, width), dtype=x_slab.dtype, device=x_slab.device)
    buf[:, :e - b] = x_slab
    parts = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf, group=group)
    x = torch.empty((rows, cols), dtype=x_slab.dtype, device=x_slab.device)
    for (lo, hi), part in zip(bounds, parts):
        x[:, lo:hi] = part[:, :hi - lo]
    return x


def _desc_array(descs: Sequence) -> "ctypes.Array":
    arr = (MatrixDesc * max(len(descs), 1))()
    for i, d in enumerate(descs):
        if isinstance(d, MatrixDesc):
            arr[i] = d
        else:       # (rows, cols, property) triple: passed through unchecked so that the planner validates it
            arr[i] = MatrixDesc(int(d[0]), int(d[1]), int(d[2]), F32 if len(d) < 4 else int(d[3]))
    return arr


class Plan:
    """Owner of a ``mom_plan_t*``; methods mirror the ``mom_plan_*`` / ``mom_equation_execute*`` calls."""

    def __init__(self, handle: int, n_chain: int, n_add: int):
        self._h = _P(handle)
        self.n_chain, self.n_add = n_chain, n_add

    def __del__(self):
        self.destroy()

    def destroy(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value and _lib is not None:   # None at interpreter exit
            _lib.mom_plan_destroy(self._h)
            self._h = _P(None)

    # ---- queries
    def flops(self) -> Tuple[int, int]:
        mul, add = ctypes.c_uint64(), ctypes.c_uint64()
        _check(_lib.mom_plan_flops(self._h, ctypes.byref(mul), ctypes.byref(add)), "mom_plan_flops")
        return mul.value, add.value

    def parenthesization(self) -> str:
        need = ctypes.c_size_t()
        st = _lib.mom_plan_parenthesization(self._h, None, 0, ctypes.byref(need))
        if st not in (OK, ERR_BUFFER_TOO_SMALL):
            _check(st, "mom_plan_parenthesization")
        buf = ctypes.create_string_buffer(need.value)
        _check(_lib.mom_plan_parenthesization(self._h, buf, need.value, None), "mom_plan_parenthesization")
        return buf.value.decode()

    def reused_products(self) -> int:
        n = ctypes.c_int32()
        _check(_lib.mom_plan_reused_products(self._h, ctypes.byref(n)), "mom_plan_reused_products")
        return n.value

    def temporaries(self) -> int:
        n = ctypes.c_int32()
        _check(_lib.mom_plan_temporaries(self._h, ctypes.byref(n)), "mom_plan_temporaries")
        return n.value

    def num_steps(self) -> int:
        n = ctypes.c_int32()
        _check(_lib.mom_plan_num_steps(self._h, ctypes.byref(n)), "mom_plan_num_steps")
        return n.value

    def step(self, i: int) -> Step:
        s = Step()
        _check(_lib.mom_plan_step(self._h, i, ctypes.byref(s)), "mom_plan_step")
        return s

    def steps(self) -> List[Step]:
        return [self.step(i) for i in range(self.num_steps())]

    def result_desc(self) -> MatrixDesc:
        d = MatrixDesc()
        _check(_lib.mom_plan_result_desc(self._h, ctypes.byref(d)), "mom_plan_result_desc")
        return d

    def workspace_bytes(self, batch: int = 1) -> int:
        b = ctypes.c_size_t()
        _check(_lib.mom_plan_workspace_bytes(self._h, batch, ctypes.byref(b)), "mom_plan_workspace_bytes")
        return b.value

    def host_staging_bytes(self, batch: int = 1) -> int:
        b = ctypes.c_size_t()
        _check(_lib.mom_plan_host_staging_bytes(self._h, batch, ctypes.byref(b)), "mom_plan_host_staging_bytes")
        return b.value

    def result_elements(self) -> int:
        """f32 entries of X as the plan writes it (rows * cols, or the packed size)."""
        n = ctypes.c_int64()
        _check(_lib.mom_plan_result_elements(self._h, ctypes.byref(n)), "mom_plan_result_elements")
        return n.value

    def host_upload_bytes(self, batch: int = 1) -> int:
        b = ctypes.c_size_t()
        _check(_lib.mom_plan_host_upload_bytes(self._h, batch, ctypes.byref(b)), "mom_plan_host_upload_bytes")
        return b.value

    def device_status(self) -> Tuple[int, int]:
        code, detail = ctypes.c_int32(), ctypes.c_int32()
        _check(_lib.mom_plan_device_status(self._h, ctypes.byref(code), ctypes.byref(detail)), "mom_plan_device_status")
        return code.value, detail.value

    def probe_wait_timeout(self, limit_ms: float, detail: int, stream: int = 0) -> None:
        """Enqueue the bounded-wait self-test: a wait nothing satisfies gives up after `limit_ms`."""
        _check(_lib.mom_probe_wait_timeout(self._h, float(limit_ms), int(detail), _P(stream)), "mom_probe_wait_timeout")

    def concurrent_steps(self) -> Tuple[int, int, int]:
        """(begin, end, join): steps [begin, end) run on the plan's side stream, step `join` waits for them; join == -1: none."""
        b, e, j = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        _check(_lib.mom_plan_concurrent_steps(self._h, ctypes.byref(b), ctypes.byref(e), ctypes.byref(j)), "mom_plan_concurrent_steps")
        return b.value, e.value, j.value

    def last_launch_count(self) -> int:
        n = ctypes.c_int32()
        _check(_lib.mom_plan_last_launch_count(self._h, ctypes.byref(n)), "mom_plan_last_launch_count")
        return n.value

    def enable_step_timing(self, enable: bool = True) -> None:
        _check(_lib.mom_plan_enable_step_timing(self._h, 1 if enable else 0), "mom_plan_enable_step_timing")

    def step_times(self, i: int) -> Tuple[float, float]:
        """(product kernel ms, pre-pass ms) of step i in the most recent execute (after a stream sync)."""
        a, b = ctypes.c_float(), ctypes.c_float()
        _check(_lib.mom_plan_step_times(self._h, i, ctypes.byref(a), ctypes.byref(b)), "mom_plan_step_times")
        return a.value, b.value

    # ---- execution (device pointers as integers)
    def execute(self, chain_ptrs: Sequence[Optional[int]], add_ptrs: Sequence[Optional[int]], out_ptr: int,
                workspace_ptr: Optional[int], workspace_bytes: int, stream: int = 0) -> None:
        _check(_lib.mom_equation_execute(self._h, _ptr_array(chain_ptrs), _ptr_array(add_ptrs) if add_ptrs else None,
                                         _P(out_ptr), _P(workspace_ptr), workspace_bytes, _P(stream)),
               "mom_equation_execute")

    def execute_batched(self, chain_ptrs, chain_strides, add_ptrs, add_strides, out_ptr: int, out_stride: int,
                        batch: int, workspace_ptr: Optional[int], workspace_bytes: int, stream: int = 0) -> None:
        cs = (ctypes.c_int64 * max(len(chain_strides), 1))(*[int(s) for s in chain_strides])
        as_ = (ctypes.c_int64 * max(len(add_strides), 1))(*[int(s) for s in add_strides])
        _check(_lib.mom_equation_execute_batched(self._h, _ptr_array(chain_ptrs), cs,
                                                 _ptr_array(add_ptrs) if add_ptrs else None, as_ if add_ptrs else None,
                                                 _P(out_ptr), out_stride, batch, _P(workspace_ptr), workspace_bytes,
                                                 _P(stream)), "mom_equation_execute_batched")

    def execute_host(self, chain_host_ptrs, add_host_ptrs, out_host_ptr: int, batch: int, staging_ptr: int,
                     staging_bytes: int, stream: int = 0) -> None:
        _check(_lib.mom_equation_execute_host(self._h, _ptr_array(chain_host_ptrs),
                                              _ptr_array(add_host_ptrs) if add_host_ptrs else None,
                                              _P(out_host_ptr), batch, _P(staging_ptr), staging_bytes, _P(stream)),
               "mom_equation_execute_host")


def mom_equation_plan(chain: Sequence, add_terms: Sequence = (), variant: int = VARIANT_3XTF32) -> Plan:
    """Plan X = prod(chain) + sum(add_terms); operands are MatrixDesc or (rows, cols, property) triples."""
    handle = _P()
    n_chain, n_add = len(chain), len(add_terms)
    st = _lib.mom_equation_plan(_desc_array(chain) if n_chain else None, n_chain,
                                _desc_array(add_terms) if n_add else None, n_add, variant, ctypes.byref(handle))
    _check(st, "mom_equation_plan")
    return Plan(handle.value, n_chain, n_add)


def mom_equation_plan_transposed(chain: Sequence, chain_transposed: Optional[Sequence], add_terms: Sequence = (),
                                 add_transposed: Optional[Sequence] = None, variant: int = VARIANT_3XTF32) -> Plan:
    """As mom_equation_plan, with per-operand Transpose flags; descriptors describe the matrices as stored."""
    handle = _P()
    n_chain, n_add = len(chain), len(add_terms)

    def flags(f, n):
        if f is None or n == 0:
            return None
        f = list(f) + [False] * (n - len(f))
        return (ctypes.c_int32 * n)(*[1 if x else 0 for x in f])
    st = _lib.mom_equation_plan_transposed(_desc_array(chain) if n_chain else None, flags(chain_transposed, n_chain), n_chain,
                                           _desc_array(add_terms) if n_add else None, flags(add_transposed, n_add), n_add,
                                           variant, ctypes.byref(handle))
    _check(st, "mom_equation_plan_transposed")
    return Plan(handle.value, n_chain, n_add)


def mom_equation_plan_stored(chain: Sequence, chain_transposed: Optional[Sequence], chain_storage: Optional[Sequence],
                             add_terms: Sequence = (), add_transposed: Optional[Sequence] = None,
                             add_storage: Optional[Sequence] = None, result_storage: int = STORAGE_DENSE,
                             variant: int = VARIANT_3XTF32) -> Plan:
    """As mom_equation_plan_transposed, with a storage (dense or packed triangle) per operand, per Add term and for X."""
    handle = _P()
    n_chain, n_add = len(chain), len(add_terms)

    def ints(f, n):
        if f is None or n == 0:
            return None
        f = list(f) + [0] * (n - len(f))
        return (ctypes.c_int32 * n)(*[int(x) for x in f])
    st = _lib.mom_equation_plan_stored(_desc_array(chain) if n_chain else None, ints(chain_transposed, n_chain), ints(chain_storage, n_chain),
                                       n_chain, _desc_array(add_terms) if n_add else None, ints(add_transposed, n_add),
                                       ints(add_storage, n_add), n_add, int(result_storage), variant, ctypes.byref(handle))
    _check(st, "mom_equation_plan_stored")
    return Plan(handle.value, n_chain, n_add)


def mom_packed_elements(rows: int, prop: int) -> int:
    """f32 entries of the packed container of a rows x rows triangle."""
    n = ctypes.c_int64()
    _check(_lib.mom_packed_elements(rows, prop, ctypes.byref(n)), "mom_packed_elements")
    return n.value


def mom_packed_row(rows: int, prop: int, row: int) -> Tuple[int, int, int]:
    """(offset, first column, end column) of row `row` in the packed container."""
    off, first, end = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    _check(_lib.mom_packed_row(rows, prop, row, ctypes.byref(off), ctypes.byref(first), ctypes.byref(end)), "mom_packed_row")
    return off.value, first.value, end.value


def mom_equation_plan_sum(chains: Sequence[Sequence], transposed: Optional[Sequence[Sequence]] = None,
                          names: Optional[Sequence[Sequence[int]]] = None, variant: int = VARIANT_3XTF32) -> Plan:
    """Plan X = sum over chains of prod(chain); the plan executes with one pointer per factor, chains flattened."""
    handle = _P()
    lengths = [len(c) for c in chains]
    flat = [d for c in chains for d in c]
    n = len(flat)
    flags = None
    if transposed is not None and n:
        rows = [list(transposed[c]) if c < len(transposed) else [] for c in range(len(chains))]
        rows = [r + [False] * (l - len(r)) for r, l in zip(rows, lengths)]
        flags = (ctypes.c_int32 * n)(*[1 if x else 0 for r in rows for x in r])
    name_arr = (ctypes.c_int32 * n)(*[int(x) for r in names for x in r]) if names is not None and n else None
    len_arr = (ctypes.c_int32 * max(len(lengths), 1))(*lengths)
    st = _lib.mom_equation_plan_sum(_desc_array(flat) if n else None, flags, name_arr, len_arr, len(lengths), variant,
                                    ctypes.byref(handle))
    _check(st, "mom_equation_plan_sum")
    return Plan(handle.value, n, 0)


EXPR_OPERAND, EXPR_MUL, EXPR_ADD, EXPR_TRANSPOSE = 0, 1, 2, 3


def mom_expression_plan(expr, operands: Sequence, variant: int = VARIANT_3XTF32) -> Plan:
    """Plan a nested expression: an operand index, ("t", e), ("mul", [e, ...]) or ("add", [e, ...]).

    The plan executes with one pointer per operand.  This function only flattens the Python value into the
    node and child arrays of the C call.
    """
    nodes: List[Tuple[int, int, int, int]] = []
    children: List[int] = []

    def emit(e) -> int:
        if isinstance(e, int):
            nodes.append((EXPR_OPERAND, e, 0, 0))
            return len(nodes) - 1
        kind = {"t": EXPR_TRANSPOSE, "mul": EXPR_MUL, "add": EXPR_ADD}.get(e[0], -1)
        kids = [emit(c) for c in ([e[1]] if e[0] == "t" else e[1])]
        nodes.append((kind, 0, len(children), len(kids)))
        children.extend(kids)
        return len(nodes) - 1

    root = emit(expr)
    node_arr = (ExprNode * len(nodes))(*[ExprNode(*n) for n in nodes])
    child_arr = (ctypes.c_int32 * max(len(children), 1))(*children)
    handle = _P()
    st = _lib.mom_expression_plan(_desc_array(operands) if len(operands) else None, len(operands), node_arr, len(nodes),
                                  child_arr, len(children), root, variant, ctypes.byref(handle))
    _check(st, "mom_expression_plan")
    return Plan(handle.value, len(operands), 0)


def mom_product_3xtf32_noalloc(m: int, n: int, k: int, pa: int, pb: int, a_ptr: int, b_ptr: int, c_ptr: int,
                               device_status_ptr: Optional[int] = None, stream: int = 0) -> None:
    """C = A*B on the tensor-core kernel using only the library's built-in scratch array (no allocation).

    For callers that cannot allocate device memory where they need the product (a plug-in inside an
    application that owns all device memory, a loop that must not hit an allocator).  Sizes beyond the
    array (2*(m*k + k*n) floats over 16 MiB) raise MomError(ERR_LIMIT).  Calls share one array per device:
    do not let two of them overlap on the GPU.
    """
    _check(_lib.mom_product_3xtf32_noalloc(m, n, k, pa, pb, _P(a_ptr), _P(b_ptr), _P(c_ptr), _P(device_status_ptr),
                                           _P(stream)), "mom_product_3xtf32_noalloc")


def mom_probe_tf32_tflops(milliseconds: float, scratch_ptr: int, stream: int = 0) -> float:
    out = ctypes.c_double()
    _check(_lib.mom_probe_tf32_tflops(milliseconds, _P(scratch_ptr), _P(stream), ctypes.byref(out)), "mom_probe_tf32_tflops")
    return out.value


def mom_probe_ffma_tflops(milliseconds: float, scratch_ptr: int, stream: int = 0) -> float:
    out = ctypes.c_double()
    _check(_lib.mom_probe_ffma_tflops(milliseconds, _P(scratch_ptr), _P(stream), ctypes.byref(out)), "mom_probe_ffma_tflops")
    return out.value
