"""TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT.

ctypes front end of the plain C oracle in ``nereus_oracle.c`` (gather the full
logical tensor, cast element by element, slice by the target plan).  Only the
tests, the smoke check and the benchmark's CPU-baseline / reference arm may
import this module; the CUDA path never does and shares no code with it.

The layout readings the oracle takes (fused per-rank QKV and gate/up blocks,
vocabulary rows, row-parallel columns, 256-byte packing, the NaN rule of the
cast) are this build's contract, not the paper's: "parity unpinned" by the
paper, pinned by the CPU tests.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nereus_oracle.c")
_LIB = os.path.join(_HERE, "libnereus_oracle.so")

BF16 = 1
FP32 = 2
QKV_GROUPED = 1
GATE_UP_INTERLEAVED = 2
VOCAB_PADDED = 4

OK = 0
ERR_ARG = -1
ERR_INDIVISIBLE = -2
ERR_UNSUPPORTED = -3
ERR_REPLICA_MISMATCH = -4
ERR_NOMEM = -5


class OracleError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"oracle: {what} failed with code {code}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, no threads)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-fPIC", "-shared",
                               _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


class _Model(ctypes.Structure):
    _fields_ = [("L", ctypes.c_int64), ("H", ctypes.c_int64), ("nq", ctypes.c_int64),
                ("nkv", ctypes.c_int64), ("F", ctypes.c_int64), ("V", ctypes.c_int64),
                ("dtype", ctypes.c_int), ("value_head", ctypes.c_int)]


class _Plan(ctypes.Structure):
    _fields_ = [("tp", ctypes.c_int), ("pp", ctypes.c_int), ("dtype", ctypes.c_int), ("layout", ctypes.c_int)]


@dataclass(frozen=True)
class Model:
    layers: int
    hidden: int
    heads: int
    kv_heads: int
    ffn: int
    vocab: int
    dtype: int = BF16
    value_head: bool = False

    def c(self) -> _Model:
        return _Model(self.layers, self.hidden, self.heads, self.kv_heads, self.ffn, self.vocab,
                      self.dtype, int(self.value_head))


@dataclass(frozen=True)
class Plan:
    tp: int
    pp: int
    dtype: int = 0  # 0 = the model's dtype
    layout: int = 0  # QKV_GROUPED | GATE_UP_INTERLEAVED | VOCAB_PADDED

    def c(self) -> _Plan:
        return _Plan(self.tp, self.pp, self.dtype, self.layout)


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, p = ctypes.c_int64, ctypes.POINTER
        L.oracle_num_logical.restype = i64
        L.oracle_num_logical.argtypes = [p(_Model)]
        L.oracle_logical_shape.argtypes = [p(_Model), i64, p(i64), p(i64)]
        L.oracle_check_plan.argtypes = [p(_Model), _Plan]
        L.oracle_num_shards.argtypes = [p(_Model), _Plan, p(i64)]
        L.oracle_shard_bytes.argtypes = [p(_Model), _Plan, i64, p(i64)]
        L.oracle_locate.argtypes = [p(_Model), _Plan, i64, i64, p(ctypes.c_int), p(i64), p(i64), p(i64),
                                    p(i64), p(i64)]
        L.oracle_part_row.restype = i64
        L.oracle_part_row.argtypes = [p(_Model), _Plan, i64, i64]
        L.oracle_rne_bf16.restype = ctypes.c_uint16
        L.oracle_rne_bf16.argtypes = [ctypes.c_uint32]
        L.oracle_rne_bf16_array.restype = None
        L.oracle_rne_bf16_array.argtypes = [ctypes.c_void_p, ctypes.c_void_p, i64]
        pp_ = p(ctypes.c_void_p)
        L.oracle_reshard_tensor_parts.argtypes = [p(_Model), _Plan, _Plan, i64, pp_, pp_]
        L.oracle_reshard_tensor.argtypes = [p(_Model), _Plan, _Plan, i64, pp_, pp_]
        L.oracle_reshard.argtypes = [p(_Model), _Plan, _Plan, pp_, pp_]
        L.oracle_reshard_replicated.argtypes = [p(_Model), _Plan, _Plan, ctypes.c_int, pp_, pp_]
        _lib = L
    return _lib


def _check(rc: int, what: str) -> None:
    if rc != OK:
        raise OracleError(rc, what)


def es(model: Model, plan: Plan) -> int:
    return 4 if (plan.dtype or model.dtype) == FP32 else 2


def num_logical(model: Model) -> int:
    m = model.c()
    return int(lib().oracle_num_logical(ctypes.byref(m)))


def logical_shape(model: Model, tid: int) -> tuple[int, int]:
    m = model.c()
    r, c = ctypes.c_int64(), ctypes.c_int64()
    _check(lib().oracle_logical_shape(ctypes.byref(m), tid, ctypes.byref(r), ctypes.byref(c)), "logical_shape")
    return r.value, c.value


def check_plan(model: Model, plan: Plan) -> int:
    m = model.c()
    return int(lib().oracle_check_plan(ctypes.byref(m), plan.c()))


def num_shards(model: Model, plan: Plan) -> int:
    m = model.c()
    n = ctypes.c_int64()
    _check(lib().oracle_num_shards(ctypes.byref(m), plan.c(), ctypes.byref(n)), "num_shards")
    return n.value


def shard_bytes(model: Model, plan: Plan, shard: int) -> int:
    m = model.c()
    n = ctypes.c_int64()
    _check(lib().oracle_shard_bytes(ctypes.byref(m), plan.c(), shard, ctypes.byref(n)), "shard_bytes")
    return n.value


@dataclass(frozen=True)
class Part:
    held: bool
    offset: int   # bytes from the start of the shard buffer
    r0: int
    nr: int
    c0: int
    nc: int


def locate(model: Model, plan: Plan, shard: int, tid: int) -> Part:
    m = model.c()
    held = ctypes.c_int()
    v = [ctypes.c_int64() for _ in range(5)]
    _check(lib().oracle_locate(ctypes.byref(m), plan.c(), shard, tid, ctypes.byref(held),
                               *[ctypes.byref(x) for x in v]), "locate")
    return Part(bool(held.value), *[x.value for x in v])


def part_row(model: Model, plan: Plan, tid: int, i: int) -> int:
    """Rows between row 0 and row i of a rank's part of logical tensor tid under the plan's layout."""
    m = model.c()
    return int(lib().oracle_part_row(ctypes.byref(m), plan.c(), tid, i))


def rne_bf16(u: int) -> int:
    return int(lib().oracle_rne_bf16(ctypes.c_uint32(u & 0xFFFFFFFF)))


def rne_bf16_array(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint32)
    out = np.empty(bits.shape, dtype=np.uint16)
    lib().oracle_rne_bf16_array(bits.ctypes.data, out.ctypes.data, bits.size)
    return out


def _ptr_array(arrs):
    n = len(arrs)
    a = (ctypes.c_void_p * n)()
    for i, x in enumerate(arrs):
        a[i] = None if x is None else x.ctypes.data
    return a


def new_shards(model: Model, plan: Plan, fill: int = 0) -> list[np.ndarray]:
    """Host shard buffers (uint8) of the sizes the plan asks for."""
    return [np.full(shard_bytes(model, plan, s), fill, dtype=np.uint8) for s in range(num_shards(model, plan))]


def reshard(model: Model, src: Plan, dst: Plan, src_bufs: list[np.ndarray],
            dst_bufs: list[np.ndarray] | None = None, fill: int = 0) -> list[np.ndarray]:
    """Whole model-stage, every logical tensor.  Buffers are uint8 numpy arrays."""
    m = model.c()
    if dst_bufs is None:
        dst_bufs = new_shards(model, dst, fill)
    for s, b in enumerate(src_bufs):
        assert b.dtype == np.uint8 and b.flags.c_contiguous and b.size >= shard_bytes(model, src, s)
    for d, b in enumerate(dst_bufs):
        assert b.dtype == np.uint8 and b.flags.c_contiguous and b.size >= shard_bytes(model, dst, d)
    _check(lib().oracle_reshard(ctypes.byref(m), src.c(), dst.c(), _ptr_array(src_bufs), _ptr_array(dst_bufs)),
           "reshard")
    return dst_bufs


def reshard_tensor(model: Model, src: Plan, dst: Plan, tid: int, src_bufs: list[np.ndarray],
                   dst_bufs: list[np.ndarray]) -> None:
    """One logical tensor, addressed by whole shard buffers."""
    m = model.c()
    _check(lib().oracle_reshard_tensor(ctypes.byref(m), src.c(), dst.c(), tid, _ptr_array(src_bufs),
                                       _ptr_array(dst_bufs)), "reshard_tensor")


def reshard_tensor_parts(model: Model, src: Plan, dst: Plan, tid: int, src_parts: list,
                         dst_parts: list) -> None:
    """One logical tensor; ``src_parts[i]`` / ``dst_parts[i]`` are uint8 arrays holding only shard i's
    part of that tensor (None where the shard does not hold it)."""
    m = model.c()
    _check(lib().oracle_reshard_tensor_parts(ctypes.byref(m), src.c(), dst.c(), tid, _ptr_array(src_parts),
                                             _ptr_array(dst_parts)), "reshard_tensor_parts")


def reshard_replicated(model: Model, src: Plan, dst: Plan, replicas: int, src_bufs: list[np.ndarray],
                       fill: int = 0) -> list[np.ndarray]:
    """k identical target units (Extend; Split into k replica units), replica-major list of shard buffers."""
    m = model.c()
    dst_bufs = [b for _ in range(replicas) for b in new_shards(model, dst, fill)]
    _check(lib().oracle_reshard_replicated(ctypes.byref(m), src.c(), dst.c(), replicas, _ptr_array(src_bufs),
                                           _ptr_array(dst_bufs)), "reshard_replicated")
    return dst_bufs


def reshard_state(model: Model, src: Plan, dst: Plan, n_opt: int, src_bufs: list[np.ndarray],
                  fill: int = 0) -> list[np.ndarray]:
    """The EMU's state (theta, omega): the parameters src -> dst, and n_opt optimizer tensors per parameter that
    are sharded exactly like the parameters (Section 5), held in fp32 on both sides and never cast.  Buffers on either side:
    parameter shards, then the shards of optimizer tensor 0, then of tensor 1, ..."""
    ns = num_shards(model, src)
    out = reshard(model, src, dst, src_bufs[:ns], fill=fill)
    m32 = Model(model.layers, model.hidden, model.heads, model.kv_heads, model.ffn, model.vocab, FP32,
                model.value_head)
    s32, d32 = Plan(src.tp, src.pp, FP32, src.layout), Plan(dst.tp, dst.pp, FP32, dst.layout)
    for k in range(n_opt):
        out += reshard(m32, s32, d32, src_bufs[ns * (1 + k):ns * (2 + k)], fill=fill)
    return out
