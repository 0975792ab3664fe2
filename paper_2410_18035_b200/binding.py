"""ctypes binding of libmilora.so: the same entry points as include/milora.h, with torch tensors
marshalled to raw device pointers.  No computation happens here; every step runs in the CUDA
library.  Importing this module fails if the library has not been built."""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmilora.so")

F32, BF16 = 0, 1
POOL_MEAN, POOL_LAST, POOL_MAX, POOL_SELFATTN = 0, 1, 2, 3
ACT_TANH, ACT_IDENTITY, ACT_RELU, ACT_GELU, ACT_RATIONAL = 0, 1, 2, 3, 4
MODULES = ("q", "k", "v", "o", "gate", "up", "down")
N_MOD = 7
GATE_NONE, GATE_PROB = 0, 1

STATUS_NAMES = {0: "MILORA_OK", 1: "MILORA_E_ARG", 2: "MILORA_E_SHAPE", 3: "MILORA_E_DTYPE",
                4: "MILORA_E_UNREGISTERED", 5: "MILORA_E_CAPACITY", 6: "MILORA_E_STATE", 7: "MILORA_E_CUDA",
                8: "MILORA_E_DEVICE_INDEX"}


class MiloraError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        self.status = status
        super().__init__(f"{what}: {STATUS_NAMES.get(status, status)}" + (f" ({detail})" if detail else ""))


class ModelDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("d_model", C.c_int), ("d_ff", C.c_int), ("d_kv", C.c_int),
                ("dtype", C.c_int), ("max_rank", C.c_int), ("max_tenants", C.c_int), ("max_requests", C.c_int),
                ("top_k", C.c_int), ("gate", C.c_int)]


class GroupLayout(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("header", "mod_offset", "mod_tile_offset", "mod_gather_offset", "seg_key",
                                           "seg_offset", "perm", "tiles", "gather_rows", "gather", "seq_tile",
                                           "total")]
    _fields_ += [("max_tiles", C.c_int), ("max_gather", C.c_int)]


class Groups(C.Structure):
    _fields_ = [("ws_dev", C.c_void_p), ("n_seq", C.c_int), ("T", C.c_int)]


class DecodeLayer(C.Structure):
    _fields_ = [("layer", C.c_int), ("groups", Groups), ("X_dev", C.c_void_p * 7), ("Y_dev", C.c_void_p * 7)]


class HostStep(C.Structure):
    _fields_ = [("layer", C.c_int), ("n_prompts", C.c_int), ("cu_prompts_host", C.c_void_p),
                ("prompt_slot_host", C.c_void_p), ("H_host", C.c_void_p), ("n_seq", C.c_int), ("T", C.c_int),
                ("cu_seq_host", C.c_void_p), ("seq_slot_host", C.c_void_p), ("X_host", C.c_void_p * 7),
                ("Y_host", C.c_void_p * 7)]


# name -> (restype, argtypes); every symbol include/milora.h declares
_VP, _I, _F = C.c_void_p, C.c_int, C.c_float
SIGNATURES = {
    "milora_create": (_I, [C.POINTER(ModelDesc), C.POINTER(_VP)]),
    "milora_destroy": (_I, [_VP]),
    "milora_status_string": (C.c_char_p, [_I]),
    "milora_last_cuda_error": (C.c_char_p, [_VP]),
    "milora_module_dims": (_I, [_VP, _I, C.POINTER(_I), C.POINTER(_I)]),
    "milora_register_adapter": (_I, [_VP, _I, _I, _I, _I, _F, _VP, _VP, _VP]),
    "milora_register_router": (_I, [_VP, _I, _I, _VP, _VP, _I, _VP, _I, C.POINTER(_F), _I, _I, _VP]),
    "milora_unregister_tenant": (_I, [_VP, _I]),
    "milora_resident_bytes": (_I, [_VP, C.POINTER(C.c_size_t)]),
    "milora_request_open": (_I, [_VP, _I, _I]),
    "milora_request_close": (_I, [_VP, _I]),
    "milora_route": (_I, [_VP, _I, _VP, _VP, _VP, _I, _I, _VP, _VP, _VP]),
    "milora_route_static": (_I, [_VP, _I, _VP, _VP, _VP, _I, _I, _VP, _VP, _VP]),
    "milora_route_table": (_I, [_VP, C.POINTER(_VP)]),
    "milora_route_table_read": (_I, [_VP, _I, _I, _VP, _VP]),
    "milora_route_table_write": (_I, [_VP, _I, _I, _VP, _VP]),
    "milora_gate_table_read": (_I, [_VP, _I, _I, _VP, _VP]),
    "milora_gate_table_write": (_I, [_VP, _I, _I, _VP, _VP]),
    "milora_group_layout": (_I, [_VP, _I, _I, C.POINTER(GroupLayout)]),
    "milora_group": (_I, [_VP, _I, _I, _VP, _VP, _I, _I, _VP, C.c_size_t, _VP]),
    "milora_set_decode_path": (_I, [_VP, _I]),
    "milora_decode_path_for": (_I, [_VP, _I, _I, C.POINTER(_I)]),
    "milora_apply_decode_layers": (_I, [_VP, C.POINTER(DecodeLayer), _I, _VP]),
    "milora_set_decode_unit_stages": (_I, [_VP, _I]),
    "milora_apply_decode": (_I, [_VP, _I, _I, _VP, _VP, C.POINTER(Groups), _VP]),
    "milora_apply_prefill": (_I, [_VP, _I, _I, _VP, _VP, C.POINTER(Groups), _VP]),
    "milora_apply_decode_multi": (_I, [_VP, _I, _I, C.POINTER(_I), C.POINTER(_VP), C.POINTER(_VP), C.POINTER(Groups), _VP]),
    "milora_apply_prefill_multi": (_I, [_VP, _I, _I, C.POINTER(_I), C.POINTER(_VP), C.POINTER(_VP), C.POINTER(Groups), _VP]),
    "milora_apply_prefill_shared": (_I, [_VP, _I, _I, C.POINTER(_I), _VP, C.POINTER(_VP), C.POINTER(Groups), _VP]),
    "milora_linear_prefill": (_I, [_VP, _I, _I, _VP, _VP, _VP, _VP, C.POINTER(Groups), _VP]),
    "milora_step_host_workspace": (_I, [_VP, C.POINTER(HostStep), C.POINTER(C.c_size_t)]),
    "milora_step_host": (_I, [_VP, C.POINTER(HostStep), _VP, C.c_size_t, _VP]),
    "milora_poll_error": (_I, [_VP, C.POINTER(_I), _VP]),
}

_lib = None


def load_library() -> C.CDLL:
    """dlopen libmilora.so and declare every prototype.  Raises if the library is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2410_18035_b200.build` "
                              "(there is no CPU fallback)")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


class Milora:
    """One library context (see include/milora.h for the meaning of every call)."""

    def __init__(self, n_layers, d_model, d_ff, d_kv, dtype, max_rank, max_tenants, max_requests, top_k=1, gate=GATE_NONE):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("the MiLoRA library needs a CUDA device; there is no CPU path")
        self.torch_dtype = {"f32": torch.float32, "bf16": torch.bfloat16}[dtype] if isinstance(dtype, str) else dtype
        code = F32 if self.torch_dtype == torch.float32 else BF16
        self.desc = ModelDesc(n_layers, d_model, d_ff, d_kv, code, max_rank, max_tenants, max_requests, top_k, gate)
        self.n_layers, self.max_requests, self.max_tenants = n_layers, max_requests, max_tenants
        self.top_k = max(1, top_k)
        h = C.c_void_p()
        self._check(self.lib.milora_create(C.byref(self.desc), C.byref(h)), "milora_create", ctx=None)
        self.h = h

    # -- helpers -------------------------------------------------------------------------
    def _check(self, status, what, ctx=True):
        if status != 0:
            detail = ""
            if status == 7 and ctx and getattr(self, "h", None):
                detail = self.lib.milora_last_cuda_error(self.h).decode()
            raise MiloraError(status, what, detail)

    def _tensor(self, t, dtype=None, name="tensor"):
        if t is None:
            return None
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous CUDA tensor")
        if dtype is not None and t.dtype != dtype:
            raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
        return t

    def close(self):
        if getattr(self, "h", None):
            self.lib.milora_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- tables --------------------------------------------------------------------------
    def module_dims(self, module):
        d1, d2 = C.c_int(), C.c_int()
        self._check(self.lib.milora_module_dims(self.h, module, C.byref(d1), C.byref(d2)), "milora_module_dims")
        return d1.value, d2.value

    def register_adapter(self, tenant, layer, module, A, B, scale, stream=None):
        self._tensor(A, self.torch_dtype, "A")
        self._tensor(B, self.torch_dtype, "B")
        d1, d2 = self.module_dims(module)
        rank = A.shape[1]
        if tuple(A.shape) != (d1, rank) or tuple(B.shape) != (rank, d2):
            raise ValueError(f"adapter shapes {tuple(A.shape)}, {tuple(B.shape)} do not fit module {module} ({d1}x{d2})")
        self._check(self.lib.milora_register_adapter(self.h, tenant, layer, module, rank, float(scale), _ptr(A), _ptr(B),
                                                     _stream(stream)), "milora_register_adapter")

    def register_router(self, tenant, layer, Wr, bias=None, pool=POOL_MEAN, Wsa=None, act=ACT_TANH, coef_a=None,
                        coef_b=None, stream=None):
        self._tensor(Wr, self.torch_dtype, "Wr")
        if tuple(Wr.shape) != (self.desc.d_model, N_MOD):
            raise ValueError("Wr must be d_model x 7")
        self._tensor(bias, torch.float32, "bias")
        self._tensor(Wsa, self.torch_dtype, "Wsa")
        coef, n_a, n_b = None, 0, 0
        if act == ACT_RATIONAL:
            a = [float(v) for v in coef_a]
            b = [float(v) for v in (coef_b if coef_b is not None else [])]
            n_a, n_b = len(a), len(b)
            coef = (C.c_float * (n_a + n_b))(*(a + b))
        self._check(self.lib.milora_register_router(self.h, tenant, layer, _ptr(Wr), _ptr(bias), pool, _ptr(Wsa), act,
                                                    coef, n_a, n_b, _stream(stream)), "milora_register_router")

    def unregister_tenant(self, tenant):
        self._check(self.lib.milora_unregister_tenant(self.h, tenant), "milora_unregister_tenant")

    def resident_bytes(self) -> int:
        out = C.c_size_t(0)
        self._check(self.lib.milora_resident_bytes(self.h, C.byref(out)), "milora_resident_bytes")
        return out.value

    def request_open(self, slot, tenant):
        self._check(self.lib.milora_request_open(self.h, slot, tenant), "milora_request_open")

    def request_close(self, slot):
        self._check(self.lib.milora_request_close(self.h, slot), "milora_request_close")

    # -- routing -------------------------------------------------------------------------
    def route(self, layer, H, cu_seqlens, seq_slot, logits_out=None, probs_out=None, stream=None):
        self._tensor(H, self.torch_dtype, "H")
        self._tensor(cu_seqlens, torch.int32, "cu_seqlens")
        self._tensor(seq_slot, torch.int32, "seq_slot")
        self._tensor(logits_out, torch.float32, "logits_out")
        self._tensor(probs_out, torch.float32, "probs_out")
        P = seq_slot.numel()
        if cu_seqlens.numel() != P + 1 or H.shape[1] != self.desc.d_model:
            raise ValueError("route: cu_seqlens must have P+1 entries and H d_model columns")
        for o in (logits_out, probs_out):
            if o is not None and o.numel() < P * N_MOD:
                raise ValueError("route: output buffers need P*7 floats")
        self._check(self.lib.milora_route(self.h, layer, _ptr(H), _ptr(cu_seqlens), _ptr(seq_slot), P, H.shape[0],
                                          _ptr(logits_out), _ptr(probs_out), _stream(stream)), "milora_route")

    def route_static(self, layer, H, cu_seqlens, seq_slot, logits_out=None, probs_out=None, stream=None):
        """milora_route_static: same as route(), with the scratch in the library's fixed device array."""
        self._tensor(H, self.torch_dtype, "H")
        self._tensor(cu_seqlens, torch.int32, "cu_seqlens")
        self._tensor(seq_slot, torch.int32, "seq_slot")
        self._tensor(logits_out, torch.float32, "logits_out")
        self._tensor(probs_out, torch.float32, "probs_out")
        P = seq_slot.numel()
        if cu_seqlens.numel() != P + 1 or H.shape[1] != self.desc.d_model:
            raise ValueError("route_static: cu_seqlens must have P+1 entries and H d_model columns")
        for o in (logits_out, probs_out):
            if o is not None and o.numel() < P * N_MOD:
                raise ValueError("route_static: output buffers need P*7 floats")
        self._check(self.lib.milora_route_static(self.h, layer, _ptr(H), _ptr(cu_seqlens), _ptr(seq_slot), P,
                                                 H.shape[0], _ptr(logits_out), _ptr(probs_out), _stream(stream)),
                    "milora_route_static")

    def route_table_ptr(self) -> int:
        p = C.c_void_p()
        self._check(self.lib.milora_route_table(self.h, C.byref(p)), "milora_route_table")
        return p.value

    def route_table_read(self, slot_begin=0, n_slots=None, stream=None):
        """[n_slots, n_layers] for top_k = 1, else [n_slots, n_layers, top_k]."""
        n_slots = self.max_requests - slot_begin if n_slots is None else n_slots
        out = torch.empty((n_slots, self.n_layers, self.top_k), dtype=torch.int32)
        self._check(self.lib.milora_route_table_read(self.h, slot_begin, n_slots, out.data_ptr(), _stream(stream)),
                    "milora_route_table_read")
        return out[:, :, 0] if self.top_k == 1 else out

    def gate_table_read(self, slot_begin=0, n_slots=None, stream=None):
        n_slots = self.max_requests - slot_begin if n_slots is None else n_slots
        out = torch.empty((n_slots, self.n_layers, self.top_k), dtype=torch.float32)
        self._check(self.lib.milora_gate_table_read(self.h, slot_begin, n_slots, out.data_ptr(), _stream(stream)),
                    "milora_gate_table_read")
        return out

    def gate_table_write(self, slot_begin, rows, stream=None):
        rows = torch.as_tensor(rows, dtype=torch.float32).contiguous().cpu()
        n_slots = rows.shape[0]
        if rows.numel() != n_slots * self.n_layers * self.top_k:
            raise ValueError("gate_table_write: rows must be [n_slots, n_layers, top_k]")
        self._check(self.lib.milora_gate_table_write(self.h, slot_begin, n_slots, rows.data_ptr(), _stream(stream)),
                    "milora_gate_table_write")

    def route_table_write(self, slot_begin, rows, stream=None):
        rows = torch.as_tensor(rows, dtype=torch.int32).contiguous().cpu()
        n_slots = rows.shape[0]
        if rows.numel() != n_slots * self.n_layers * self.top_k:
            raise ValueError("route_table_write: rows must be [n_slots, n_layers] (or [n_slots, n_layers, top_k])")
        self._check(self.lib.milora_route_table_write(self.h, slot_begin, n_slots, rows.data_ptr(), _stream(stream)),
                    "milora_route_table_write")

    # -- grouping ------------------------------------------------------------------------
    def group_layout(self, n_seq, T) -> GroupLayout:
        lay = GroupLayout()
        self._check(self.lib.milora_group_layout(self.h, n_seq, T, C.byref(lay)), "milora_group_layout")
        return lay

    def alloc_group_ws(self, n_layers, n_seq, T, device=None):
        lay = self.group_layout(n_seq, T)
        return torch.empty((n_layers, lay.total), dtype=torch.int32, device=device or "cuda")

    def group(self, layer_begin, n_layers, cu_seqlens, seq_slot, n_seq, T, ws, stream=None):
        self._tensor(cu_seqlens, torch.int32, "cu_seqlens")
        self._tensor(seq_slot, torch.int32, "seq_slot")
        self._tensor(ws, torch.int32, "ws")
        if seq_slot is not None and seq_slot.numel() < n_seq:
            raise ValueError("group: seq_slot shorter than n_seq")
        if cu_seqlens is not None and cu_seqlens.numel() < n_seq + 1:
            raise ValueError("group: cu_seqlens shorter than n_seq + 1")
        if ws.dim() != 2 or ws.shape[0] < n_layers:
            raise ValueError("group: ws must be [n_layers, stride]")
        self._check(self.lib.milora_group(self.h, layer_begin, n_layers, _ptr(cu_seqlens), _ptr(seq_slot), n_seq, T,
                                          _ptr(ws), ws.shape[1], _stream(stream)), "milora_group")

    def groups(self, ws_layer, n_seq, T) -> Groups:
        """Descriptor of one layer's block (a row of the tensor alloc_group_ws returned)."""
        self._tensor(ws_layer, torch.int32, "ws_layer")
        return Groups(ws_layer.data_ptr(), n_seq, T)

    # -- apply ---------------------------------------------------------------------------
    def _xy(self, module, X, Y, T):
        d1, d2 = self.module_dims(module)
        self._tensor(X, self.torch_dtype, "X")
        self._tensor(Y, self.torch_dtype, "Y")
        if X.shape[0] < T or Y.shape[0] < T or X.shape[1] != d1 or Y.shape[1] != d2:
            raise ValueError(f"apply: X/Y shapes {tuple(X.shape)}/{tuple(Y.shape)} do not fit module {module} with T={T}")

    def set_decode_path(self, path):
        """milora_set_decode_path: 0 / "auto", 1 / "cluster" (one launch), 2 / "split" (two streaming launches),
        3 / "stream" (the persistent kernel of apply_decode_layers)."""
        code = {"auto": 0, "cluster": 1, "split": 2, "stream": 3}.get(path, path)
        self._check(self.lib.milora_set_decode_path(self.h, int(code)), "milora_set_decode_path")

    def decode_path_for(self, n_seq, T):
        """milora_decode_path_for: 1 (cluster, one launch) or 2 (split, two launches) for such a batch."""
        out = C.c_int(0)
        self._check(self.lib.milora_decode_path_for(self.h, n_seq, T, C.byref(out)), "milora_decode_path_for")
        return out.value

    def set_decode_unit_stages(self, unit_stages):
        self._check(self.lib.milora_set_decode_unit_stages(self.h, int(unit_stages)), "milora_set_decode_unit_stages")

    def decode_layers(self, entries) -> "C.Array":
        """Marshals [(layer, groups, {module: (X, Y)}), ...] into the milora_decode_layer array that
        apply_decode_layers takes (build it once for a decode loop over fixed buffers)."""
        arr = (DecodeLayer * len(entries))()
        for i, (layer, groups, sites) in enumerate(entries):
            arr[i].layer = layer
            arr[i].groups = groups
            for m, (X, Y) in sites.items():
                self._xy(m, X, Y, groups.T)
                arr[i].X_dev[m] = X.data_ptr()
                arr[i].Y_dev[m] = Y.data_ptr()
        return arr

    def apply_decode_layers(self, layers, stream=None):
        """milora_apply_decode_layers on an array made by decode_layers()."""
        self._check(self.lib.milora_apply_decode_layers(self.h, layers, len(layers), _stream(stream)),
                    "milora_apply_decode_layers")

    def apply_decode(self, layer, module, X, Y, groups: Groups, stream=None):
        self._xy(module, X, Y, groups.T)
        self._check(self.lib.milora_apply_decode(self.h, layer, module, _ptr(X), _ptr(Y), C.byref(groups),
                                                 _stream(stream)), "milora_apply_decode")

    def apply_prefill(self, layer, module, X, Y, groups: Groups, stream=None):
        self._xy(module, X, Y, groups.T)
        self._check(self.lib.milora_apply_prefill(self.h, layer, module, _ptr(X), _ptr(Y), C.byref(groups),
                                                  _stream(stream)), "milora_apply_prefill")

    def _multi(self, fn, what, layer, modules, Xs, Ys, groups, stream):
        n = len(modules)
        for m, X, Y in zip(modules, Xs, Ys):
            self._xy(m, X, Y, groups.T)
        mods = (C.c_int * n)(*modules)
        xs = (C.c_void_p * n)(*[X.data_ptr() for X in Xs])
        ys = (C.c_void_p * n)(*[Y.data_ptr() for Y in Ys])
        self._check(fn(self.h, layer, n, mods, xs, ys, C.byref(groups), _stream(stream)), what)

    def apply_decode_multi(self, layer, modules, Xs, Ys, groups: Groups, stream=None):
        self._multi(self.lib.milora_apply_decode_multi, "milora_apply_decode_multi", layer, modules, Xs, Ys, groups, stream)

    def apply_prefill_multi(self, layer, modules, Xs, Ys, groups: Groups, stream=None):
        self._multi(self.lib.milora_apply_prefill_multi, "milora_apply_prefill_multi", layer, modules, Xs, Ys, groups, stream)

    def apply_prefill_shared(self, layer, modules, X, Ys, groups: Groups, stream=None):
        """milora_apply_prefill_shared: the listed modules all read X ([T, d1]); Ys[i] is module i's output."""
        n = len(modules)
        for m, Y in zip(modules, Ys):
            self._xy(m, X, Y, groups.T)
        mods = (C.c_int * n)(*modules)
        ys = (C.c_void_p * n)(*[Y.data_ptr() for Y in Ys])
        self._check(self.lib.milora_apply_prefill_shared(self.h, layer, n, mods, _ptr(X), ys, C.byref(groups),
                                                         _stream(stream)), "milora_apply_prefill_shared")

    def linear_prefill(self, layer, module, X, Wt, Y, groups: Groups, bias=None, stream=None):
        """milora_linear_prefill: Y = X W + b + LoRA term of the routed prompt rows; Wt is [d2, d1]."""
        self._xy(module, X, Y, groups.T)
        d1, d2 = self.module_dims(module)
        self._tensor(Wt, self.torch_dtype, "Wt")
        self._tensor(bias, self.torch_dtype, "bias")
        if tuple(Wt.shape) != (d2, d1) or (bias is not None and bias.numel() != d2):
            raise ValueError(f"linear_prefill: Wt must be [{d2}, {d1}] and bias [{d2}]")
        self._check(self.lib.milora_linear_prefill(self.h, layer, module, _ptr(X), _ptr(Wt), _ptr(bias), _ptr(Y),
                                                   C.byref(groups), _stream(stream)), "milora_linear_prefill")

    # -- one step from host buffers ------------------------------------------------------
    def make_host_step(self, layer, cu_prompts, prompt_slot, H, cu_seq, seq_slot, T, Xs, Ys) -> HostStep:
        """Descriptor of milora_step_host.  All tensors are HOST tensors (pinned for asynchronous copies):
        cu_prompts / prompt_slot / H describe the prompts to route (None: no routing); cu_seq / seq_slot the
        step's sequences; Xs / Ys are dicts module -> [T, d1] / [T, d2] host tensors.  The caller keeps the
        tensors alive until the stream has been synchronised."""
        def host(t, dtype, name):
            if t is None:
                return None
            if t.is_cuda or not t.is_contiguous() or t.dtype != dtype:
                raise ValueError(f"{name} must be a contiguous host tensor of dtype {dtype}")
            return t
        st = HostStep()
        st.layer = layer
        st.n_prompts = 0 if prompt_slot is None else prompt_slot.numel()
        st.cu_prompts_host = _ptr(host(cu_prompts, torch.int32, "cu_prompts"))
        st.prompt_slot_host = _ptr(host(prompt_slot, torch.int32, "prompt_slot"))
        st.H_host = _ptr(host(H, self.torch_dtype, "H"))
        st.n_seq = 0 if seq_slot is None else seq_slot.numel()
        st.T = T
        st.cu_seq_host = _ptr(host(cu_seq, torch.int32, "cu_seq"))
        st.seq_slot_host = _ptr(host(seq_slot, torch.int32, "seq_slot"))
        for m in range(N_MOD):
            x, y = Xs.get(m), Ys.get(m)
            if (x is None) != (y is None):
                raise ValueError("X and Y must be given together")
            if x is not None:
                d1, d2 = self.module_dims(m)
                if tuple(x.shape) != (T, d1) or tuple(y.shape) != (T, d2):
                    raise ValueError(f"host step: module {m} needs X [{T},{d1}] and Y [{T},{d2}]")
            st.X_host[m] = _ptr(host(x, self.torch_dtype, "X"))
            st.Y_host[m] = _ptr(host(y, self.torch_dtype, "Y"))
        return st

    def step_host_workspace(self, step: HostStep) -> int:
        n = C.c_size_t(0)
        self._check(self.lib.milora_step_host_workspace(self.h, C.byref(step), C.byref(n)), "milora_step_host_workspace")
        return n.value

    def step_host(self, step: HostStep, workspace, stream=None):
        if not workspace.is_cuda or workspace.dtype != torch.uint8:
            raise ValueError("workspace must be a CUDA uint8 tensor")
        self._check(self.lib.milora_step_host(self.h, C.byref(step), workspace.data_ptr(), workspace.numel(),
                                              _stream(stream)), "milora_step_host")

    def poll_error(self, stream=None) -> int:
        flag = C.c_int(0)
        st = self.lib.milora_poll_error(self.h, C.byref(flag), _stream(stream))
        if st not in (0, 8):
            self._check(st, "milora_poll_error")
        return flag.value
