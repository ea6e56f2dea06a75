"""ctypes binding of the C ABI declared in ``include/edg_moe.h``: argument marshalling only.

Every function has the name and argument order of its C counterpart.  Buffers are torch tensors
(device or pinned), numpy arrays (host) or raw integer addresses; torch is used for memory and
streams only.  A non-zero status raises :class:`EdgError`.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

__all__ = [
    "EdgError", "LayerDesc", "Lora", "StoreStats", "HotStats", "CopyEngine", "make_copy_engine", "Store", "F32", "F16", "BF16", "LIB_PATH",
    "make_desc", "make_lora", "version", "check_desc", "record_bytes", "pack_expert", "unpack_expert",
    "ffn_workspace_bytes", "workspace_status", "set_trace_buffer", "prerouter_topk", "prerouter_topk_tokens", "softmax_topk_rows", "sigmoid_group_topk_rows", "prerouter_mlp_topk",
    "moe_expert_ffn_int4_lora", "moe_expert_ffn_int4_lora_static", "moe_layer_decode", "stage_experts_to_slots",
    "moe_layer_decode_dependent", "stack_decode_token", "next_hidden_state", "EXPORTS",
]

F32, F16, BF16 = 0, 1, 2
_ERR = {-1: "EDG_E_INVAL", -2: "EDG_E_SHAPE", -3: "EDG_E_SLOTS", -4: "EDG_E_RANGE", -5: "EDG_E_CUDA",
        -6: "EDG_E_TIMEOUT", -7: "EDG_E_WORKSPACE"}

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libedgmoe.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2609_18063_b200.build` "
        "(nvcc, sm_100a). There is no fallback path.")
_lib = C.CDLL(LIB_PATH)


class EdgError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        msg = f"{what}: {_ERR.get(code, code)}"
        if code == -5:
            msg += f" ({_lib.edg_last_cuda_error_string().decode()})"
        super().__init__(msg)


class LayerDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("H", "I", "E", "K", "group", "rank", "n_adapters", "n_slots",
                                          "pre_dtype", "out_dtype")] + [("lora_scale", C.c_float)]


class Lora(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("A_gate", "B_gate", "A_up", "B_up", "A_down", "B_down")]


class HotStats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("hits", "misses", "admitted", "bytes_direct")]


_ENG_FN = {
    "copy_h2d": C.CFUNCTYPE(C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p),
    "fill": C.CFUNCTYPE(C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_size_t, C.c_void_p),
    "event_create": C.CFUNCTYPE(C.c_int32, C.c_void_p, C.POINTER(C.c_void_p)),
    "event_destroy": C.CFUNCTYPE(C.c_int32, C.c_void_p, C.c_void_p),
    "event_record": C.CFUNCTYPE(C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p),
    "stream_wait_event": C.CFUNCTYPE(C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p),
    "event_synchronize": C.CFUNCTYPE(C.c_int32, C.c_void_p, C.c_void_p),
    "stream_synchronize": C.CFUNCTYPE(C.c_int32, C.c_void_p, C.c_void_p),
    "host_alloc": C.CFUNCTYPE(C.c_int32, C.c_void_p, C.POINTER(C.c_void_p), C.c_size_t),
    "host_free": C.CFUNCTYPE(C.c_int32, C.c_void_p, C.c_void_p),
}


class CopyEngine(C.Structure):
    """edg_copy_engine: ``ctx`` plus ten callbacks, in the header's order."""
    _fields_ = [("ctx", C.c_void_p)] + [(n, t) for n, t in _ENG_FN.items()]


def make_copy_engine(obj) -> CopyEngine:
    """Wraps an object that has the ten methods of edg_copy_engine (same arguments, ctx first).
    The returned struct keeps the callbacks alive through its ``_keep`` attribute."""
    fns = {n: t(getattr(obj, n)) for n, t in _ENG_FN.items()}
    eng = CopyEngine(None, *[fns[n] for n in _ENG_FN])
    eng._keep = (obj, fns)
    return eng


class StoreStats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("stage_calls", "hits", "misses", "bytes_copied", "table_updates")]


_P = C.c_void_p
_D = C.POINTER(LayerDesc)
_SIG = {
    "edg_version": ([], C.c_int32),
    "edg_last_cuda_error": ([], C.c_int32),
    "edg_last_cuda_error_string": ([], C.c_char_p),
    "edg_check_desc": ([_D], C.c_int32),
    "edg_record_bytes": ([_D, C.POINTER(C.c_size_t)], C.c_int32),
    "edg_pack_expert": ([_D] + [_P] * 10, C.c_int32),
    "edg_unpack_expert": ([_D] + [_P] * 10, C.c_int32),
    "edg_ffn_workspace_bytes": ([_D, C.c_int32, C.POINTER(C.c_size_t)], C.c_int32),
    "edg_workspace_status": ([_P, _P, C.POINTER(C.c_int32)], C.c_int32),
    "edg_set_trace_buffer": ([_P], C.c_int32),
    "prerouter_topk": ([_D, _P, _P, C.c_int32, _P, _P, _P, _P, _P], C.c_int32),
    "prerouter_topk_tokens": ([_D, _P, _P, C.c_int32, _P, _P, _P, _P], C.c_int32),
    "softmax_topk_rows": ([_D, _P, C.c_int32, _P, _P, _P], C.c_int32),
    "sigmoid_group_topk_rows": ([_P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_float, _P, _P, _P, _P], C.c_int32),
    "prerouter_mlp_topk": ([_D, _P, _P, _P, _P, C.c_int32, _P, _P, _P, _P], C.c_int32),
    "moe_layer_decode_dependent": ([_P, C.c_int32, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, C.c_float, _P, C.c_size_t, _P], C.c_int32),
    "edg_store_create": ([_D, C.c_int32, C.POINTER(_P), _P, _P, C.POINTER(Lora), _P, C.POINTER(_P)], C.c_int32),
    "edg_store_create_ex": ([_D, C.c_int32, C.POINTER(_P), _P, _P, C.POINTER(Lora), _P, C.POINTER(CopyEngine), C.POINTER(_P)], C.c_int32),
    "edg_store_destroy": ([_P], C.c_int32),
    "edg_store_load_whole_layer": ([_P, C.c_int32, _P], C.c_int32),
    "edg_store_set_mlp_head": ([_P, C.c_int32, _P], C.c_int32),
    "edg_store_reset_feedback": ([_P, C.c_int32], C.c_int32),
    "edg_store_set_hot": ([_P, C.c_int32, C.c_int32], C.c_int32),
    "edg_store_set_shared_expert": ([_P, C.c_int32, _P, C.POINTER(Lora)], C.c_int32),
    "edg_store_get_hot_stats": ([_P, C.POINTER(HotStats)], C.c_int32),
    "edg_store_get_stats": ([_P, C.POINTER(StoreStats)], C.c_int32),
    "edg_store_set_chaining": ([_P, C.c_int32], C.c_int32),
    "edg_store_snapshot": ([_P, C.c_int32, _P, _P], C.c_int32),
    "edg_store_wait_staged": ([_P, C.c_int32, _P], C.c_int32),
    "edg_store_time_waits": ([_P, C.c_int32], C.c_int32),
    "edg_store_exposed_wait_ms": ([_P, C.POINTER(C.c_double), C.POINTER(C.c_int64)], C.c_int32),
    "edg_stack_decode_token": ([_P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, C.c_size_t, _P, C.c_int32, C.POINTER(C.c_int32)], C.c_int32),
    "edg_next_hidden_state": ([_D, _P, _P, _P, C.c_float, _P], C.c_int32),
    "edg_store_mark_computed": ([_P, C.c_int32, _P], C.c_int32),
    "stage_experts_to_slots": ([_P, C.c_int32, _P, C.c_int32, _P, C.POINTER(C.c_int32)], C.c_int32),
    "moe_expert_ffn_int4_lora": ([_D, _P, _P, C.c_int32, _P, _P, _P, _P, C.POINTER(Lora), _P, _P, C.c_size_t, _P], C.c_int32),
    "moe_expert_ffn_int4_lora_static": ([_D, _P, _P, _P, _P, _P, _P, C.POINTER(Lora), _P, _P], C.c_int32),
    "moe_layer_decode": ([_P, C.c_int32, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, C.c_size_t, _P], C.c_int32),
}
EXPORTS = tuple(_SIG)
for _name, (_args, _res) in _SIG.items():
    _fn = getattr(_lib, _name)          # AttributeError here = the library lacks a declared symbol
    _fn.argtypes = _args
    _fn.restype = _res


def _check(code: int, what: str) -> None:
    if code != 0:
        raise EdgError(code, what)


def _ptr(buf) -> Optional[int]:
    """Address of a torch tensor, a numpy array, a raw int, or None."""
    if buf is None:
        return None
    if isinstance(buf, int):
        return buf
    if isinstance(buf, np.ndarray):
        if not buf.flags["C_CONTIGUOUS"]:
            raise ValueError("numpy buffer must be C-contiguous")
        return buf.ctypes.data
    if hasattr(buf, "data_ptr"):
        if not buf.is_contiguous():
            raise ValueError("tensor must be contiguous")
        return buf.data_ptr()
    raise TypeError(f"cannot take the address of {type(buf)!r}")


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


_DT = {"f32": F32, "f16": F16, "bf16": BF16}


def make_desc(cfg=None, *, out_dtype="f32", **kw) -> LayerDesc:
    """Descriptor from a workload config object (fields H, I, E, K, group, rank, n_adapters,
    n_slots, pre_dtype, lora_scale) and/or keyword overrides."""
    vals = {}
    if cfg is not None:
        for n in ("H", "I", "E", "K", "group", "rank", "n_adapters", "n_slots", "lora_scale", "pre_dtype"):
            vals[n] = getattr(cfg, n)
    vals.update(kw)
    pre = vals.get("pre_dtype", "f16")
    d = LayerDesc()
    for n in ("H", "I", "E", "K", "group", "rank", "n_adapters", "n_slots"):
        setattr(d, n, int(vals[n]))
    d.pre_dtype = _DT[pre] if isinstance(pre, str) else int(pre)
    d.out_dtype = _DT[out_dtype] if isinstance(out_dtype, str) else int(out_dtype)
    d.lora_scale = float(vals.get("lora_scale", 1.0))
    return d


def make_lora(A_gate, B_gate, A_up, B_up, A_down, B_down) -> Lora:
    """The struct only carries addresses: the caller keeps the tensors alive."""
    return Lora(*[_ptr(t) for t in (A_gate, B_gate, A_up, B_up, A_down, B_down)])


def version() -> int:
    return _lib.edg_version()


def check_desc(desc: LayerDesc) -> int:
    return _lib.edg_check_desc(C.byref(desc))


def record_bytes(desc: LayerDesc) -> int:
    n = C.c_size_t()
    _check(_lib.edg_record_bytes(C.byref(desc), C.byref(n)), "edg_record_bytes")
    return n.value


def _canon(tensors):
    """proj -> (codes u8, scales f16, zeros f16)  ->  nine contiguous host arrays."""
    out = []
    for proj in ("gate", "up", "down"):
        c, s, z = tensors[proj]
        out += [np.ascontiguousarray(c, dtype=np.uint8),
                np.ascontiguousarray(np.asarray(s, dtype=np.float16).view(np.uint16)),
                np.ascontiguousarray(np.asarray(z, dtype=np.float16).view(np.uint16))]
    return out


def pack_expert(desc: LayerDesc, tensors, record=None) -> np.ndarray:
    """Canonical tensors of one expert -> kernel record (numpy uint8, or written into `record`)."""
    arrs = _canon(tensors)
    shapes = {"gate": (desc.I, desc.H), "up": (desc.I, desc.H), "down": (desc.H, desc.I)}
    for i, proj in enumerate(("gate", "up", "down")):
        n, kd = shapes[proj]
        if arrs[3 * i].shape != (n, kd // 2) or arrs[3 * i + 1].shape != (n, kd // desc.group) \
                or arrs[3 * i + 2].shape != (n, kd // desc.group):
            raise ValueError(f"{proj}: tensor shapes do not match the descriptor")
    if record is None:
        record = np.empty(record_bytes(desc), dtype=np.uint8)
    _check(_lib.edg_pack_expert(C.byref(desc), *[_ptr(a) for a in arrs], _ptr(record)), "edg_pack_expert")
    return record


def unpack_expert(desc: LayerDesc, record):
    shapes = {"gate": (desc.I, desc.H), "up": (desc.I, desc.H), "down": (desc.H, desc.I)}
    arrs = []
    for proj in ("gate", "up", "down"):
        n, kd = shapes[proj]
        arrs += [np.empty((n, kd // 2), np.uint8), np.empty((n, kd // desc.group), np.uint16),
                 np.empty((n, kd // desc.group), np.uint16)]
    _check(_lib.edg_unpack_expert(C.byref(desc), _ptr(record), *[_ptr(a) for a in arrs]), "edg_unpack_expert")
    return {p: (arrs[3 * i], arrs[3 * i + 1].view(np.float16), arrs[3 * i + 2].view(np.float16))
            for i, p in enumerate(("gate", "up", "down"))}


def ffn_workspace_bytes(desc: LayerDesc, T: int = 1) -> int:
    n = C.c_size_t()
    _check(_lib.edg_ffn_workspace_bytes(C.byref(desc), T, C.byref(n)), "edg_ffn_workspace_bytes")
    return n.value


def workspace_status(workspace, stream=None) -> int:
    st = C.c_int32()
    _check(_lib.edg_workspace_status(_ptr(workspace), _stream(stream), C.byref(st)), "edg_workspace_status")
    return st.value


def set_trace_buffer(dev_buffer) -> None:
    """Phase timestamps of the batch-1 layer kernel into `dev_buffer` (uint64 [CTAs][16]); None = off."""
    _check(_lib.edg_set_trace_buffer(_ptr(dev_buffer)), "edg_set_trace_buffer")


def prerouter_topk(desc, W_pre, s, n_heads, inds, gates, logits_opt=None, stream=None, inds_host_mirror_opt=None) -> None:
    _check(_lib.prerouter_topk(C.byref(desc), _ptr(W_pre), _ptr(s), n_heads, _ptr(inds), _ptr(gates),
                               _ptr(logits_opt), _ptr(inds_host_mirror_opt), _stream(stream)), "prerouter_topk")


def prerouter_topk_tokens(desc, W_pre, s, T, inds, gates, logits_opt=None, stream=None) -> None:
    _check(_lib.prerouter_topk_tokens(C.byref(desc), _ptr(W_pre), _ptr(s), T, _ptr(inds), _ptr(gates),
                                      _ptr(logits_opt), _stream(stream)), "prerouter_topk_tokens")


class MlpHead(C.Structure):
    _fields_ = [("W1", _P), ("b1", _P), ("W2", _P), ("b2", _P), ("W_res", _P), ("width", C.c_int32)]


def prerouter_mlp_topk(desc, W1, b1, W2, b2, W_res, width, s, cur_inds, prev_inds, n_heads, inds, gates,
                       logits_opt=None, stream=None) -> None:
    head = MlpHead(_ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(W_res), int(width))
    _check(_lib.prerouter_mlp_topk(C.byref(desc), C.byref(head), _ptr(s), _ptr(cur_inds), _ptr(prev_inds), n_heads,
                                   _ptr(inds), _ptr(gates), _ptr(logits_opt), _stream(stream)), "prerouter_mlp_topk")


def sigmoid_group_topk_rows(logits, T, E, K, n_groups, keep_groups, scale, bias, inds, gates, stream=None) -> None:
    _check(_lib.sigmoid_group_topk_rows(_ptr(logits), T, E, K, n_groups, keep_groups, float(scale), _ptr(bias),
                                        _ptr(inds), _ptr(gates), _stream(stream)), "sigmoid_group_topk_rows")


def softmax_topk_rows(desc, logits, T, inds, gates, stream=None) -> None:
    _check(_lib.softmax_topk_rows(C.byref(desc), _ptr(logits), T, _ptr(inds), _ptr(gates), _stream(stream)),
           "softmax_topk_rows")


def moe_expert_ffn_int4_lora(desc, slot_pool, slot_table, T, slots, experts, gates, x, lora, y,
                             workspace, workspace_bytes=None, stream=None) -> None:
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(_lib.moe_expert_ffn_int4_lora(C.byref(desc), _ptr(slot_pool), _ptr(slot_table), T, _ptr(slots),
                                         _ptr(experts), _ptr(gates), _ptr(x),
                                         None if lora is None else C.byref(lora), _ptr(y), _ptr(workspace),
                                         workspace_bytes, _stream(stream)), "moe_expert_ffn_int4_lora")


def moe_expert_ffn_int4_lora_static(desc, slot_pool, slot_table, slots, experts, gates, x, lora, y, stream=None) -> None:
    """Batch-1 FFN without a caller-provided workspace: for hosts that may not allocate device
    memory.  The scratch is a fixed array inside the library; see the header for the rules
    (first call per device before any stream capture; overlapping calls race)."""
    _check(_lib.moe_expert_ffn_int4_lora_static(C.byref(desc), _ptr(slot_pool), _ptr(slot_table), _ptr(slots),
                                                _ptr(experts), _ptr(gates), _ptr(x),
                                                None if lora is None else C.byref(lora), _ptr(y), _stream(stream)),
           "moe_expert_ffn_int4_lora_static")


class Store:
    """Owner of an ``edg_store`` handle.  Keeps references to the caller's buffers alive."""

    def __init__(self, desc: LayerDesc, host_layers: Sequence, dev_slots, dev_tables,
                 loras: Optional[Sequence[Lora]] = None, copy_stream=None, engine: Optional[CopyEngine] = None):
        self.desc = desc
        self.n_layers = len(host_layers)
        self._keep = (list(host_layers), dev_slots, dev_tables, loras, copy_stream, engine)
        ptrs = (_P * self.n_layers)(*[_ptr(h) for h in host_layers])
        lor = None
        if loras is not None:
            lor = (Lora * self.n_layers)(*loras)
        h = _P()
        if engine is None:
            _check(_lib.edg_store_create(C.byref(desc), self.n_layers, ptrs, _ptr(dev_slots), _ptr(dev_tables),
                                         lor, _stream(copy_stream), C.byref(h)), "edg_store_create")
        else:                       # a caller's engine: streams are whatever that engine understands
            _check(_lib.edg_store_create_ex(C.byref(desc), self.n_layers, ptrs, _ptr(dev_slots), _ptr(dev_tables),
                                            lor, copy_stream, C.byref(engine), C.byref(h)), "edg_store_create_ex")
        self._foreign = engine is not None
        self.handle = h

    def close(self) -> None:
        if getattr(self, "handle", None):
            _check(_lib.edg_store_destroy(self.handle), "edg_store_destroy")
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_chaining(self, enable) -> None:
        """False / 0: off (default); True / 1: chain a step when the one before it is still in flight;
        2: chain whenever the buffers line up."""
        _check(_lib.edg_store_set_chaining(self.handle, int(enable)), "edg_store_set_chaining")

    def stats(self) -> dict:
        s = StoreStats()
        _check(_lib.edg_store_get_stats(self.handle, C.byref(s)), "edg_store_get_stats")
        return {n: getattr(s, n) for n, _ in StoreStats._fields_}

    def snapshot(self, layer: int):
        eos = np.empty(self.desc.n_slots, np.int32)
        soe = np.empty(self.desc.E, np.int32)
        _check(_lib.edg_store_snapshot(self.handle, layer, _ptr(eos), _ptr(soe)), "edg_store_snapshot")
        return eos, soe

    def set_mlp_head(self, layer: int, W1=None, b1=None, W2=None, b2=None, W_res=None, width: int = 0) -> None:
        """The full prerouter head of a layer (tensors of ONE head; the caller keeps them alive); W1 None removes it."""
        if W1 is None:
            _check(_lib.edg_store_set_mlp_head(self.handle, layer, None), "edg_store_set_mlp_head")
            return
        self._keep = self._keep + (W1, b1, W2, b2, W_res)
        head = MlpHead(_ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(W_res), int(width))
        _check(_lib.edg_store_set_mlp_head(self.handle, layer, C.byref(head)), "edg_store_set_mlp_head")

    def reset_feedback(self, layer: int) -> None:
        _check(_lib.edg_store_reset_feedback(self.handle, layer), "edg_store_reset_feedback")

    def load_whole_layer(self, layer: int, host_layer=None) -> None:
        _check(_lib.edg_store_load_whole_layer(self.handle, layer, _ptr(host_layer)), "edg_store_load_whole_layer")

    def set_shared_expert(self, layer: int, dev_record, lora: Optional[Lora] = None) -> None:
        """The caller keeps `dev_record` and the adapter's tensors alive."""
        self._keep = self._keep + (dev_record, lora)
        _check(_lib.edg_store_set_shared_expert(self.handle, layer, _ptr(dev_record), None if lora is None else C.byref(lora)),
               "edg_store_set_shared_expert")

    def set_hot(self, enable: bool = True, admit_after: int = 1) -> None:
        _check(_lib.edg_store_set_hot(self.handle, int(bool(enable)), int(admit_after)), "edg_store_set_hot")

    def hot_stats(self) -> dict:
        s = HotStats()
        _check(_lib.edg_store_get_hot_stats(self.handle, C.byref(s)), "edg_store_get_hot_stats")
        return {n: getattr(s, n) for n, _ in HotStats._fields_}

    def _st(self, stream):
        return stream if self._foreign else _stream(stream)

    def wait_staged(self, layer: int, stream=None) -> None:
        _check(_lib.edg_store_wait_staged(self.handle, layer, self._st(stream)), "edg_store_wait_staged")

    def time_waits(self, enable: bool) -> None:
        _check(_lib.edg_store_time_waits(self.handle, int(bool(enable))), "edg_store_time_waits")

    def exposed_wait_ms(self):
        """(ms the compute streams waited for staging copies since the last call, number of waits)."""
        ms, n = C.c_double(), C.c_int64()
        _check(_lib.edg_store_exposed_wait_ms(self.handle, C.byref(ms), C.byref(n)), "edg_store_exposed_wait_ms")
        return ms.value, n.value

    def mark_computed(self, layer: int, stream=None) -> None:
        _check(_lib.edg_store_mark_computed(self.handle, layer, self._st(stream)), "edg_store_mark_computed")


def stage_experts_to_slots(store: Store, layer: int, inds_host, n: Optional[int] = None):
    """Returns (slots int32 [n], n_miss)."""
    inds = np.ascontiguousarray(inds_host, dtype=np.int32)
    n = len(inds) if n is None else n
    slots = np.empty(max(n, 1), np.int32)
    miss = C.c_int32()
    _check(_lib.stage_experts_to_slots(store.handle, layer, _ptr(inds), n, _ptr(slots), C.byref(miss)),
           "stage_experts_to_slots")
    return slots[:n], miss.value


def moe_layer_decode(store: Store, layer, x, inds_cur, gates_cur, W_pre_next, inds_next, gates_next,
                     logits_next_opt, y, workspace, workspace_bytes=None, stream=None,
                     inds_next_host_mirror_opt=None) -> None:
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(_lib.moe_layer_decode(store.handle, layer, _ptr(x), _ptr(inds_cur), _ptr(gates_cur), _ptr(W_pre_next),
                                 _ptr(inds_next), _ptr(gates_next), _ptr(logits_next_opt),
                                 _ptr(inds_next_host_mirror_opt), _ptr(y),
                                 _ptr(workspace), workspace_bytes, _stream(stream)), "moe_layer_decode")


def stack_decode_token(store: Store, x, inds_cur, gates_cur, W_pre, inds_next, gates_next, logits_next_opt,
                       mirror_cur, mirror_next, y, workspace, workspace_bytes=None, stream=None, prefetch=True) -> int:
    """edg_stack_decode_token; returns the number of experts copied for this token."""
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    miss = C.c_int32()
    _check(_lib.edg_stack_decode_token(store.handle, _ptr(x), _ptr(inds_cur), _ptr(gates_cur), _ptr(W_pre),
                                       _ptr(inds_next), _ptr(gates_next), _ptr(logits_next_opt), _ptr(mirror_cur),
                                       _ptr(mirror_next), _ptr(y), _ptr(workspace), workspace_bytes, _stream(stream),
                                       int(bool(prefetch)), C.byref(miss)), "edg_stack_decode_token")
    return miss.value


def next_hidden_state(desc, x, y, x_next, eps=1e-6, stream=None) -> None:
    _check(_lib.edg_next_hidden_state(C.byref(desc), _ptr(x), _ptr(y), _ptr(x_next), float(eps), _stream(stream)),
           "edg_next_hidden_state")


def moe_layer_decode_dependent(store: Store, layer, x, inds_cur, gates_cur, W_pre_next, inds_next, gates_next,
                               logits_next_opt, y, x_next, workspace, eps=1e-6, workspace_bytes=None, stream=None,
                               inds_next_host_mirror_opt=None) -> None:
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(_lib.moe_layer_decode_dependent(store.handle, layer, _ptr(x), _ptr(inds_cur), _ptr(gates_cur), _ptr(W_pre_next),
                                           _ptr(inds_next), _ptr(gates_next), _ptr(logits_next_opt),
                                           _ptr(inds_next_host_mirror_opt), _ptr(y), _ptr(x_next), float(eps),
                                           _ptr(workspace), workspace_bytes, _stream(stream)), "moe_layer_decode_dependent")
