"""Thin ctypes binding of ``libnereus.so`` (the C ABI of ``include/nereus.h``), same names, argument
marshalling only: every step of the reshard runs inside the CUDA library.  Importing this module loads the
library and raises if it has not been built (``python -m paper_2609_34645_b200.build``); there is no CPU
fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnereus.so")

BF16 = 1
FP32 = 2
DTYPES = {"bf16": BF16, "fp32": FP32}
QKV_GROUPED = 1
GATE_UP_INTERLEAVED = 2
VOCAB_PADDED = 4

OK = 0
ERR_ARG, ERR_INDIVISIBLE, ERR_UNSUPPORTED, ERR_ALIAS = -1, -2, -3, -4
ERR_CUDA, ERR_NOMEM, ERR_MISMATCH, ERR_ALIGN = -5, -6, -7, -8
ERR_TOO_LARGE = -9
ERR_INFEASIBLE = -10
ERR_TABLE = -11
ERR_TOO_SMALL = -12
GENERATION, INFERENCE, TRAINING = 0, 1, 2
OP_SPLIT, OP_DESTROY, OP_EXTEND, OP_MERGE = 0, 1, 2, 3
STATIC_MAX_RECTS = 4096
DEV_OK, DEV_BOUNDS, DEV_TIMEOUT = 0, 1, 2

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_34645_b200.build` "
                      "(nvcc, sm_100a).  The reshard has no CPU fallback.")
_lib = ctypes.CDLL(LIB_PATH)


class NereusError(RuntimeError):
    def __init__(self, code: int, what: str):
        msg = _lib.nereus_strerror(code).decode()
        if code == ERR_CUDA:
            msg += f" (cudaError {_lib.nereus_last_cuda_error()})"
        super().__init__(f"{what}: {msg} [{code}]")
        self.code = code


class Plan(ctypes.Structure):
    """nereus_plan_t: (tp, pp, dtype, layout); dtype 0 = the descriptor's; layout = QKV_GROUPED |
    GATE_UP_INTERLEAVED."""
    _fields_ = [("tp", ctypes.c_int), ("pp", ctypes.c_int), ("dtype", ctypes.c_int), ("layout", ctypes.c_int)]

    def __init__(self, tp: int, pp: int, dtype: int = 0, layout: int = 0):
        super().__init__(tp, pp, dtype, layout)

    def __repr__(self):
        return f"Plan(tp={self.tp}, pp={self.pp}, dtype={self.dtype}, layout={self.layout})"


class Rect(ctypes.Structure):
    """nereus_rect_t."""
    _fields_ = [("src_buf", ctypes.c_int32), ("dst_buf", ctypes.c_int32), ("level", ctypes.c_int32),
                ("cast", ctypes.c_int32), ("src_off", ctypes.c_uint64), ("dst_off", ctypes.c_uint64),
                ("src_pitch", ctypes.c_uint64), ("dst_pitch", ctypes.c_uint64), ("rows", ctypes.c_uint64),
                ("width_bytes_src", ctypes.c_uint64), ("width_bytes_dst", ctypes.c_uint64),
                ("replicas", ctypes.c_int32), ("replica_stride", ctypes.c_int32)]


class Horizon(ctypes.Structure):
    """nereus_horizon_t: the EMA of crossing intervals H_x."""
    _fields_ = [("h_steps", ctypes.c_double), ("weight", ctypes.c_double), ("observed", ctypes.c_int)]

    def __init__(self, weight: float = 0.5):
        super().__init__()
        _ck(_lib.nereus_horizon_init(ctypes.byref(self), weight), "nereus_horizon_init")

    def crossing(self, interval_steps: float) -> float:
        _ck(_lib.nereus_horizon_crossing(ctypes.byref(self), interval_steps), "nereus_horizon_crossing")
        return self.h_steps


class BlockTrace(ctypes.Structure):
    """nereus_block_trace_t: one block of a traced run."""
    _fields_ = [("begin_ns", ctypes.c_uint64), ("end_ns", ctypes.c_uint64), ("tiles", ctypes.c_uint32),
                ("block", ctypes.c_uint32)]


class PrimInfo(ctypes.Structure):
    """nereus_prim_t."""
    _fields_ = [(n, ctypes.c_int32) for n in ("op", "stage", "n_src", "n_dst", "n_deps", "n_resource_deps",
                                              "order", "level")]


_vp, _i, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
_P = ctypes.POINTER
_SIGS = {
    "nereus_model_desc": [_i, _i, _i, _i, _i, _i, _i, _P(_vp)],
    "nereus_model_desc_set_value_head": [_vp, _i],
    "nereus_model_desc_destroy": [_vp],
    "nereus_plan_check": [_vp, Plan],
    "nereus_plan_num_shards": [_vp, Plan, _P(_i)],
    "nereus_plan_shard_bytes": [_vp, Plan, _i, _P(_sz)],
    "nereus_model_num_tensors": [_vp, _P(_i)],
    "nereus_plan_tensor_slice": [_vp, Plan, _i, _i, _P(_sz), _P(_sz), _P(_sz), _P(_i)],
    "nereus_transition_compile": [_vp, Plan, Plan, _P(_vp)],
    "nereus_transition_compile_replicated": [_vp, Plan, Plan, _i, _P(_vp)],
    "nereus_transition_compile_state": [_vp, Plan, Plan, _i, _P(_vp)],
    "nereus_transition_fuse": [_P(_vp), _i, _i, _P(_vp)],
    "nereus_transition_destroy": [_vp],
    "nereus_transition_num_buffers": [_vp, _P(_i), _P(_i)],
    "nereus_transition_buffer_bytes": [_vp, _i, _i, _P(_sz)],
    "nereus_transition_bytes": [_vp, _P(_sz), _P(_sz)],
    "nereus_transition_num_rects": [_vp, _P(_i)],
    "nereus_transition_get_rect": [_vp, _i, _P(Rect)],
    "nereus_transition_num_tiles": [_vp, _P(ctypes.c_uint64), _P(_i)],
    "nereus_transition_get_tiles": [_vp, ctypes.c_uint64, ctypes.c_uint64, _P(Rect)],
    "nereus_transition_tune": [_vp, _i, _i, _i, _i],
    "nereus_transition_prepare": [_vp],
    "nereus_transition_launch_info": [_vp, _P(_i), _P(_i), _P(_i), _P(_i)],
    "nereus_transition_run": [_vp, _P(_vp), _P(_vp), _vp],
    "nereus_transition_run_sized": [_vp, _P(_vp), _P(_sz), _P(_vp), _P(_sz), _vp],
    "nereus_transition_status": [_vp, _P(_i)],
    "nereus_transition_launches": [_vp, _P(ctypes.c_uint64)],
    "nereus_transition_trace": [_vp, _i],
    "nereus_transition_trace_read": [_vp, _P(BlockTrace), _i, _P(_i)],
    "nereus_last_cuda_error": [],
    "nereus_dag_create": [_P(_vp)],
    "nereus_dag_destroy": [_vp],
    "nereus_dag_add_stage": [_vp, _i, ctypes.c_uint64, _P(_i)],
    "nereus_dag_add_unit": [_vp, _i, _i, _i, _i, _P(_i)],
    "nereus_dag_plan": [_vp, ctypes.c_uint64],
    "nereus_dag_num_units": [_vp, _P(_i)],
    "nereus_dag_unit": [_vp, _i, _P(_i), _P(_i), _P(_i), _P(_i), _i],
    "nereus_dag_num_prims": [_vp, _P(_i)],
    "nereus_dag_prim": [_vp, _i, _P(PrimInfo)],
    "nereus_dag_prim_lists": [_vp, _i, _P(_i), _P(_i), _P(_i), _P(_i)],
    "nereus_dag_lower": [_vp, _P(_vp), _i, _P(_vp)],
    "nereus_transition_estimate": [_vp, ctypes.c_double, ctypes.c_double, _P(ctypes.c_double)],
    "nereus_admit": [ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double, _i,
                     _P(_i), _P(ctypes.c_double)],
    "nereus_horizon_init": [_P(Horizon), ctypes.c_double],
    "nereus_horizon_crossing": [_P(Horizon), ctypes.c_double],
    "nereus_transition_run_static": [_vp, _P(_vp), _P(_vp), _vp],
    "nereus_static_status": [_P(_i)],
    "nereus_transition_validate": [_vp],
    "nereus_debug_set_rect": [_vp, _i, _P(Rect)],
}
for _name, _args in _SIGS.items():
    _f = getattr(_lib, _name)          # AttributeError here = the library does not export a declared symbol
    _f.argtypes = _args
    _f.restype = _i
_lib.nereus_strerror.argtypes = [_i]
_lib.nereus_strerror.restype = ctypes.c_char_p
EXPORTS = sorted(list(_SIGS) + ["nereus_strerror"])


def _ck(rc: int, what: str) -> None:
    if rc != OK:
        raise NereusError(rc, what)


class ModelDesc:
    """nereus_model_desc(layers, hidden, heads, kv_heads, ffn, vocab, dtype)."""

    def __init__(self, layers, hidden, heads, kv_heads, ffn, vocab, dtype=BF16, value_head=False):
        self._h = _vp()
        _ck(_lib.nereus_model_desc(layers, hidden, heads, kv_heads, ffn, vocab, dtype, ctypes.byref(self._h)),
            "nereus_model_desc")
        if value_head:
            self.set_value_head(1)

    def set_value_head(self, out_dim=1):
        _ck(_lib.nereus_model_desc_set_value_head(self._h, out_dim), "nereus_model_desc_set_value_head")

    def plan_check(self, plan: Plan) -> int:
        return _lib.nereus_plan_check(self._h, plan)

    def num_shards(self, plan: Plan) -> int:
        n = _i()
        _ck(_lib.nereus_plan_num_shards(self._h, plan, ctypes.byref(n)), "nereus_plan_num_shards")
        return n.value

    def shard_bytes(self, plan: Plan, shard: int) -> int:
        n = _sz()
        _ck(_lib.nereus_plan_shard_bytes(self._h, plan, shard, ctypes.byref(n)), "nereus_plan_shard_bytes")
        return n.value

    def shard_sizes(self, plan: Plan) -> list:
        return [self.shard_bytes(plan, s) for s in range(self.num_shards(plan))]

    def num_tensors(self) -> int:
        n = _i()
        _ck(_lib.nereus_model_num_tensors(self._h, ctypes.byref(n)), "nereus_model_num_tensors")
        return n.value

    def tensor_slice(self, plan: Plan, shard: int, tensor_id: int):
        """(offset, rows, cols, replicated) of a stored tensor in a shard; rows = cols = 0 if not held."""
        off, r, c, rep = _sz(), _sz(), _sz(), _i()
        _ck(_lib.nereus_plan_tensor_slice(self._h, plan, shard, tensor_id, ctypes.byref(off), ctypes.byref(r),
                                          ctypes.byref(c), ctypes.byref(rep)), "nereus_plan_tensor_slice")
        return off.value, r.value, c.value, bool(rep.value)

    def compile(self, src: Plan, dst: Plan) -> "Transition":
        h = _vp()
        _ck(_lib.nereus_transition_compile(self._h, src, dst, ctypes.byref(h)), "nereus_transition_compile")
        return Transition(h)

    def compile_replicated(self, src: Plan, dst: Plan, replicas: int) -> "Transition":
        """k identical destination units, every source byte read once (Extend when src == dst)."""
        h = _vp()
        _ck(_lib.nereus_transition_compile_replicated(self._h, src, dst, replicas, ctypes.byref(h)),
            "nereus_transition_compile_replicated")
        return Transition(h)

    def compile_state(self, src: Plan, dst: Plan, n_opt: int) -> "Transition":
        """Parameters plus n_opt fp32 optimizer tensors per parameter, all in one table."""
        h = _vp()
        _ck(_lib.nereus_transition_compile_state(self._h, src, dst, n_opt, ctypes.byref(h)),
            "nereus_transition_compile_state")
        return Transition(h)

    def close(self):
        if self._h:
            _lib.nereus_model_desc_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Transition:
    """A compiled transition handle (nereus_transition_t)."""

    def __init__(self, handle):
        self._h = handle

    @staticmethod
    def fuse(parts, chained=False) -> "Transition":
        arr = (_vp * len(parts))(*[p._h for p in parts])
        h = _vp()
        _ck(_lib.nereus_transition_fuse(arr, len(parts), int(chained), ctypes.byref(h)), "nereus_transition_fuse")
        return Transition(h)

    def num_buffers(self):
        a, b = _i(), _i()
        _ck(_lib.nereus_transition_num_buffers(self._h, ctypes.byref(a), ctypes.byref(b)),
            "nereus_transition_num_buffers")
        return a.value, b.value

    def buffer_bytes(self, is_dst: bool, index: int) -> int:
        n = _sz()
        _ck(_lib.nereus_transition_buffer_bytes(self._h, int(is_dst), index, ctypes.byref(n)),
            "nereus_transition_buffer_bytes")
        return n.value

    def bytes(self):
        r, w = _sz(), _sz()
        _ck(_lib.nereus_transition_bytes(self._h, ctypes.byref(r), ctypes.byref(w)), "nereus_transition_bytes")
        return r.value, w.value

    def rects(self) -> list:
        n = _i()
        _ck(_lib.nereus_transition_num_rects(self._h, ctypes.byref(n)), "nereus_transition_num_rects")
        out = []
        for k in range(n.value):
            r = Rect()
            _ck(_lib.nereus_transition_get_rect(self._h, k, ctypes.byref(r)), "nereus_transition_get_rect")
            out.append(r)
        return out

    def validate(self) -> int:
        """nereus_transition_validate: the host-side check of the task table; returns the error code."""
        return _lib.nereus_transition_validate(self._h)

    def debug_set_rect(self, index: int, rect: Rect) -> None:
        """Test hook: overwrite one task of a table that has not been uploaded, unchecked."""
        _ck(_lib.nereus_debug_set_rect(self._h, index, ctypes.byref(rect)), "nereus_debug_set_rect")

    def prepare_raw(self) -> int:
        return _lib.nereus_transition_prepare(self._h)

    def num_tiles(self):
        t, l = ctypes.c_uint64(), _i()
        _ck(_lib.nereus_transition_num_tiles(self._h, ctypes.byref(t), ctypes.byref(l)), "nereus_transition_num_tiles")
        return t.value, l.value

    def tiles(self, first=0, count=None) -> list:
        """The tiling one run walks, each tile as the task it amounts to (nereus_transition_get_tiles)."""
        if count is None:
            count = self.num_tiles()[0] - first
        arr = (Rect * max(1, count))()
        _ck(_lib.nereus_transition_get_tiles(self._h, first, count, arr), "nereus_transition_get_tiles")
        return list(arr[:count])

    def tune(self, tile_bytes=0, ctas_per_sm=0, threads=0, variant=0):
        _ck(_lib.nereus_transition_tune(self._h, tile_bytes, ctas_per_sm, threads, variant), "nereus_transition_tune")

    def launch_info(self) -> dict:
        v, tb, g, th = _i(), _i(), _i(), _i()
        _ck(_lib.nereus_transition_launch_info(self._h, ctypes.byref(v), ctypes.byref(tb), ctypes.byref(g),
                                               ctypes.byref(th)), "nereus_transition_launch_info")
        return {"kernel": {1: "nereus_walk_vec", 2: "nereus_walk_ring", 3: "nereus_walk_once"}[v.value], "tile_bytes": tb.value,
                "grid": g.value, "threads": th.value}

    def estimate(self, gbytes_per_s: float, setup_seconds: float = 0.0) -> float:
        """L_tran in seconds from the table's bytes, a bandwidth and a set-up time."""
        out = ctypes.c_double()
        _ck(_lib.nereus_transition_estimate(self._h, gbytes_per_s, setup_seconds, ctypes.byref(out)),
            "nereus_transition_estimate")
        return out.value

    def prepare(self):
        _ck(_lib.nereus_transition_prepare(self._h), "nereus_transition_prepare")

    @staticmethod
    def pointer_array(ptrs):
        return (_vp * len(ptrs))(*ptrs)

    def run(self, src_ptrs, dst_ptrs, stream=0):
        """src_ptrs / dst_ptrs: sequences of device addresses (ints) or ready ctypes arrays; stream: a
        cudaStream_t as an int (e.g. torch.cuda.current_stream().cuda_stream)."""
        if not isinstance(src_ptrs, ctypes.Array):
            src_ptrs = self.pointer_array(src_ptrs)
        if not isinstance(dst_ptrs, ctypes.Array):
            dst_ptrs = self.pointer_array(dst_ptrs)
        _ck(_lib.nereus_transition_run(self._h, src_ptrs, dst_ptrs, _vp(stream)), "nereus_transition_run")

    def run_raw(self, src_ptrs, dst_ptrs, stream=0) -> int:
        """Like run() but returns the error code instead of raising."""
        if not isinstance(src_ptrs, ctypes.Array):
            src_ptrs = self.pointer_array(src_ptrs)
        if not isinstance(dst_ptrs, ctypes.Array):
            dst_ptrs = self.pointer_array(dst_ptrs)
        return _lib.nereus_transition_run(self._h, src_ptrs, dst_ptrs, _vp(stream))

    def run_sized_raw(self, src_ptrs, src_sizes, dst_ptrs, dst_sizes, stream=0) -> int:
        """nereus_transition_run_sized: run() with the lengths of the caller's buffers; returns the error code."""
        sp, dp = self.pointer_array(src_ptrs), self.pointer_array(dst_ptrs)
        ss, ds = (_sz * len(src_sizes))(*src_sizes), (_sz * len(dst_sizes))(*dst_sizes)
        return _lib.nereus_transition_run_sized(self._h, sp, ss, dp, ds, _vp(stream))

    def run_static(self, src_ptrs, dst_ptrs, stream=0):
        """nereus_transition_run_static: the same transition without any device allocation, for callers
        whose memory pool owns the whole GPU.  At most STATIC_MAX_RECTS tasks; calls that overlap on the
        device race on the shared table; refused while the stream is being captured; its device status is
        read with static_status()."""
        if not isinstance(src_ptrs, ctypes.Array):
            src_ptrs = self.pointer_array(src_ptrs)
        if not isinstance(dst_ptrs, ctypes.Array):
            dst_ptrs = self.pointer_array(dst_ptrs)
        _ck(_lib.nereus_transition_run_static(self._h, src_ptrs, dst_ptrs, _vp(stream)),
            "nereus_transition_run_static")

    def run_static_raw(self, src_ptrs, dst_ptrs, stream=0) -> int:
        if not isinstance(src_ptrs, ctypes.Array):
            src_ptrs = self.pointer_array(src_ptrs)
        if not isinstance(dst_ptrs, ctypes.Array):
            dst_ptrs = self.pointer_array(dst_ptrs)
        return _lib.nereus_transition_run_static(self._h, src_ptrs, dst_ptrs, _vp(stream))

    def status(self) -> int:
        s = _i()
        _ck(_lib.nereus_transition_status(self._h, ctypes.byref(s)), "nereus_transition_status")
        return s.value

    def trace(self, enable=True) -> None:
        """Switches the per-block trace on or off (drops the device copy of the table)."""
        _ck(_lib.nereus_transition_trace(self._h, int(enable)), "nereus_transition_trace")

    def trace_read(self) -> list:
        """[(block, begin_ns, end_ns, tiles)] of the last run; the caller has synchronised."""
        cap = max(1, self.launch_info()["grid"])
        arr, n = (BlockTrace * cap)(), _i()
        _ck(_lib.nereus_transition_trace_read(self._h, arr, cap, ctypes.byref(n)), "nereus_transition_trace_read")
        return [(r.block, r.begin_ns, r.end_ns, r.tiles) for r in arr[:n.value]]

    def launches(self) -> int:
        n = ctypes.c_uint64()
        _ck(_lib.nereus_transition_launches(self._h, ctypes.byref(n)), "nereus_transition_launches")
        return n.value

    def close(self):
        if self._h:
            _lib.nereus_transition_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Dag:
    """Transition DAG over EMU primitives (nereus_dag_*)."""

    def __init__(self):
        self._h = _vp()
        _ck(_lib.nereus_dag_create(ctypes.byref(self._h)), "nereus_dag_create")

    def add_stage(self, kind: int, state_bytes: int) -> int:
        s = _i()
        _ck(_lib.nereus_dag_add_stage(self._h, kind, state_bytes, ctypes.byref(s)), "nereus_dag_add_stage")
        return s.value

    def add_unit(self, stage: int, is_target: bool, tp: int, pp: int, gpus) -> None:
        arr = (_i * len(gpus))(*gpus)
        if len(gpus) != tp * pp:
            raise ValueError("a unit needs tp*pp GPUs")
        _ck(_lib.nereus_dag_add_unit(self._h, stage, int(is_target), tp, pp, arr), "nereus_dag_add_unit")

    def plan(self, gpu_capacity: int = 0) -> None:
        _ck(_lib.nereus_dag_plan(self._h, gpu_capacity), "nereus_dag_plan")

    def units(self) -> list:
        n = _i()
        _ck(_lib.nereus_dag_num_units(self._h, ctypes.byref(n)), "nereus_dag_num_units")
        out = []
        for u in range(n.value):
            st, tp, pp = _i(), _i(), _i()
            _ck(_lib.nereus_dag_unit(self._h, u, ctypes.byref(st), ctypes.byref(tp), ctypes.byref(pp), None, 0),
                "nereus_dag_unit")
            g = (_i * (tp.value * pp.value))()
            _ck(_lib.nereus_dag_unit(self._h, u, ctypes.byref(st), ctypes.byref(tp), ctypes.byref(pp), g, len(g)),
                "nereus_dag_unit")
            out.append((st.value, tp.value, pp.value, tuple(g)))
        return out

    def prims(self) -> list:
        """[{op, stage, src, dst, deps, resource_deps, order, level}] by primitive index."""
        n = _i()
        _ck(_lib.nereus_dag_num_prims(self._h, ctypes.byref(n)), "nereus_dag_num_prims")
        out = []
        for k in range(n.value):
            info = PrimInfo()
            _ck(_lib.nereus_dag_prim(self._h, k, ctypes.byref(info)), "nereus_dag_prim")
            a = [(_i * max(1, c))() for c in (info.n_src, info.n_dst, info.n_deps, info.n_resource_deps)]
            _ck(_lib.nereus_dag_prim_lists(self._h, k, *a), "nereus_dag_prim_lists")
            out.append({"op": info.op, "stage": info.stage, "src": tuple(a[0][:info.n_src]),
                        "dst": tuple(a[1][:info.n_dst]), "deps": set(a[2][:info.n_deps]),
                        "resource_deps": set(a[3][:info.n_resource_deps]), "order": info.order,
                        "level": info.level})
        return out

    def lower(self, descs) -> "Transition":
        """One task table for the whole DAG; descs[m] is the ModelDesc of model-stage m."""
        arr = (_vp * len(descs))(*[d._h for d in descs])
        h = _vp()
        _ck(_lib.nereus_dag_lower(self._h, arr, len(descs), ctypes.byref(h)), "nereus_dag_lower")
        return Transition(h)

    def close(self):
        if self._h:
            _lib.nereus_dag_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def admit(l_tran, l_step_current, l_step_target, gamma=0.5, h_x=1.0, urgent=False):
    """Eq. 2: returns (admitted, payback period in steps)."""
    a, pb = _i(), ctypes.c_double()
    _ck(_lib.nereus_admit(l_tran, l_step_current, l_step_target, gamma, h_x, int(urgent), ctypes.byref(a),
                          ctypes.byref(pb)), "nereus_admit")
    return bool(a.value), pb.value


def static_status() -> int:
    """nereus_static_status: device status of the static runs on the current device (reading clears it)."""
    s = _i()
    _ck(_lib.nereus_static_status(ctypes.byref(s)), "nereus_static_status")
    return s.value


def strerror(code: int) -> str:
    return _lib.nereus_strerror(code).decode()
