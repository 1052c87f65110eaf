"""Thin ctypes binding of libmix.so: argument marshalling only.

Every step of the hook runs in the CUDA kernels behind the C ABI (include/mix.h); this
module turns torch tensors into device pointers and checks return codes.  There is no CPU
fallback: if the library is missing or cannot be loaded, importing callers fail loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

from . import _build

MIX_PROBE, MIX_STEER, MIX_SAE, MIX_PROJECT, MIX_ROUTER = 1, 2, 3, 4, 5
MIX_ACT_SIGMOID, MIX_ACT_SOFTMAX, MIX_ACT_NONE = 0, 1, 2
MIX_SAE_RELU, MIX_SAE_JUMPRELU, MIX_SAE_TOPK = 0, 1, 2
MIX_EDIT_CLAMP, MIX_EDIT_ABLATE = 0, 1
MIX_GATE_GE, MIX_GATE_LT = 0, 1
MIX_STATUS_BAD_SLOT, MIX_STATUS_BAD_GROUP, MIX_STATUS_WAIT_TIMEOUT, MIX_STATUS_TOPK_GENERAL = 1, 2, 4, 8
MIX_FLAG_ENCODE_SIMT = 1
MIX_FLAG_RETILE_W_ENC = 2
MIX_FLAG_TEST_STALL_ENCODE = 4
MIX_FLAG_SAE_EDIT_ONLY = 8
MIX_FLAG_SLOT_CHAINS = 16
MIX_FLAG_FP8_W_ENC = 32
MIX_FLAG_FP8_ACT = 64

EXPORTS = [
    "mix_create", "mix_destroy", "mix_last_error", "mix_register_sae_weights", "mix_unregister_sae_weights",
    "mix_register_app", "mix_unregister_app", "mix_set_gate", "mix_set_chain", "mix_update_steer_alpha", "mix_update_sae_edits",
    "mix_set_slot_map", "mix_set_request_map", "mix_set_feature_out", "mix_apply", "mix_apply_conditional", "mix_apply_router", "mix_get_status",
    "mix_launches_per_apply", "mix_set_stage_events", "mix_debug_workspace", "mix_sae_apply_static",
    "mix_bench_param_update", "mix_set_pdl_mask", "mix_debug_phase_clocks",
]


class MixConfig(C.Structure):
    _fields_ = [("d_model", C.c_int), ("T_max", C.c_int), ("n_slots_max", C.c_int), ("n_groups_max", C.c_int),
                ("C_max", C.c_int), ("k_max", C.c_int), ("r_max", C.c_int), ("d_sae_max", C.c_longlong),
                ("flags", C.c_uint)]


class MixProbe(C.Structure):
    _fields_ = [("n_classes", C.c_int), ("act", C.c_int), ("W", C.c_void_p), ("b", C.c_void_p)]


class MixSteer(C.Structure):
    _fields_ = [("v", C.c_void_p), ("alpha", C.c_float)]


class MixRouter(C.Structure):
    _fields_ = [("n_experts", C.c_int), ("delta", C.c_void_p)]


class MixSaeWeights(C.Structure):
    _fields_ = [("d_sae", C.c_longlong), ("act", C.c_int), ("k", C.c_int), ("W_enc", C.c_void_p),
                ("b_enc", C.c_void_p), ("theta", C.c_void_p), ("W_dec", C.c_void_p), ("b_dec", C.c_void_p),
                ("center_input", C.c_int), ("W_enc_scale", C.c_void_p)]


class MixSaeApp(C.Structure):
    _fields_ = [("group", C.c_int), ("n_edit", C.c_int), ("idx", C.c_void_p), ("val", C.c_void_p),
                ("mode", C.c_void_p), ("add_error", C.c_int)]


class MixError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("mix error %d: %s" % (code, msg))
        self.code = code


_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Load libmix.so (built in-tree).  Raises if it is absent: there is no other path."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or _build.LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError("libmix.so not found at %s; run __graft_entry__.build() first" % path)
    lib = C.CDLL(path)
    vp, ci = C.c_void_p, C.c_int
    lib.mix_create.argtypes = [C.POINTER(vp), C.POINTER(MixConfig)]
    lib.mix_destroy.argtypes = [vp]
    lib.mix_last_error.argtypes = [vp]
    lib.mix_last_error.restype = C.c_char_p
    lib.mix_register_sae_weights.argtypes = [vp, ci, C.POINTER(MixSaeWeights), vp]
    lib.mix_unregister_sae_weights.argtypes = [vp, ci, vp]
    lib.mix_register_app.argtypes = [vp, ci, ci, vp, vp]
    lib.mix_unregister_app.argtypes = [vp, ci, vp]
    lib.mix_set_gate.argtypes = [vp, ci, vp, ci, ci, ci, C.c_float, vp]
    lib.mix_set_chain.argtypes = [vp, ci, ci, vp]
    lib.mix_update_steer_alpha.argtypes = [vp, ci, C.c_float, vp]
    lib.mix_update_sae_edits.argtypes = [vp, ci, ci, vp, vp, vp, vp]
    lib.mix_set_slot_map.argtypes = [vp, vp, ci, ci, vp]
    lib.mix_set_request_map.argtypes = [vp, vp, ci, vp, ci, ci, vp]
    lib.mix_set_feature_out.argtypes = [vp, vp, vp, vp]
    lib.mix_apply.argtypes = [vp, vp, ci, vp, vp]
    lib.mix_apply_conditional.argtypes = [vp, vp, ci, vp, vp]
    lib.mix_apply_router.argtypes = [vp, vp, ci, ci, vp]
    lib.mix_get_status.argtypes = [vp, C.POINTER(C.c_uint), vp]
    lib.mix_launches_per_apply.argtypes = [vp]
    lib.mix_set_stage_events.argtypes = [vp, C.POINTER(vp)]
    lib.mix_set_pdl_mask.argtypes = [ci]
    lib.mix_bench_param_update.argtypes = [vp, ci, C.POINTER(C.c_float), C.POINTER(C.c_float), vp]
    lib.mix_sae_apply_static.argtypes = [vp, ci, ci, C.POINTER(MixSaeWeights), C.POINTER(MixSaeApp), vp, vp, vp,
                                         C.c_char_p, ci]
    lib.mix_debug_workspace.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(C.c_longlong), C.POINTER(ci)]
    lib.mix_debug_phase_clocks.argtypes = [vp, C.POINTER(C.c_ulonglong)]
    for name in EXPORTS:
        if name != "mix_last_error":
            getattr(lib, name).restype = ci
    if path == _build.LIB_PATH:
        _lib = lib
    return lib


def set_pdl_mask(mask: int) -> int:
    """Which launches use programmatic dependent launch (see mix_set_pdl_mask); returns the previous mask."""
    return int(load_library().mix_set_pdl_mask(int(mask)))


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    h = stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)
    return h or None


class Mix:
    """One hook context on the current CUDA device (same names as the C ABI)."""

    def __init__(self, d_model, T_max, n_slots_max, n_groups_max=0, C_max=1, k_max=0, r_max=0, d_sae_max=0,
                 flags=0):
        if not torch.cuda.is_available():
            raise RuntimeError("mix needs a CUDA device (sm_100a); there is no CPU path")
        self.lib = load_library()
        self.cfg = MixConfig(d_model, T_max, n_slots_max, n_groups_max, C_max, k_max, r_max, d_sae_max, flags)
        self.ctx = C.c_void_p()
        rc = self.lib.mix_create(C.byref(self.ctx), C.byref(self.cfg))
        if rc != 0:
            raise MixError(rc, "mix_create failed")
        self._keep = {}          # borrowed weights must outlive their registration

    def _check(self, rc):
        if rc != 0:
            raise MixError(rc, self.lib.mix_last_error(self.ctx).decode())

    def destroy(self):
        if self.ctx:
            self.lib.mix_destroy(self.ctx)
            self.ctx = C.c_void_p()
            self._keep.clear()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def register_sae_weights(self, group, d_sae, act, k, W_enc, b_enc, W_dec, theta=None, b_dec=None,
                             center_input=False, w_scale=None, stream=None):
        """W_enc: bf16 [d_sae, d]; in a MIX_FLAG_FP8_W_ENC context uint8 E4M3 codes with w_scale fp32 [d_sae]."""
        w = MixSaeWeights(int(d_sae), int(act), int(k), _ptr(W_enc), _ptr(b_enc), _ptr(theta), _ptr(W_dec),
                          _ptr(b_dec), int(bool(center_input)), _ptr(w_scale))
        self._check(self.lib.mix_register_sae_weights(self.ctx, group, C.byref(w), _stream(stream)))
        self._keep[("g", group)] = (W_enc, b_enc, W_dec, theta, b_dec, w_scale)

    def unregister_sae_weights(self, group, stream=None):
        self._check(self.lib.mix_unregister_sae_weights(self.ctx, group, _stream(stream)))

    def register_probe(self, slot, W, b, act, stream=None):
        d = MixProbe(int(W.shape[0]), int(act), _ptr(W), _ptr(b))
        self._check(self.lib.mix_register_app(self.ctx, slot, MIX_PROBE, C.byref(d), _stream(stream)))
        self._keep[("a", slot)] = (W, b)

    def register_steer(self, slot, v, alpha, stream=None):
        d = MixSteer(_ptr(v), float(alpha))
        self._check(self.lib.mix_register_app(self.ctx, slot, MIX_STEER, C.byref(d), _stream(stream)))
        self._keep[("a", slot)] = (v,)

    def register_project(self, slot, r, beta, stream=None):
        d = MixSteer(_ptr(r), float(beta))          # mix_project has the layout of mix_steer: (pointer, float)
        self._check(self.lib.mix_register_app(self.ctx, slot, MIX_PROJECT, C.byref(d), _stream(stream)))
        self._keep[("a", slot)] = (r,)

    def register_router(self, slot, delta, stream=None):
        assert delta.dtype == torch.float32 and delta.dim() == 1
        d = MixRouter(int(delta.numel()), _ptr(delta))
        self._check(self.lib.mix_register_app(self.ctx, slot, MIX_ROUTER, C.byref(d), _stream(stream)))
        self._keep[("a", slot)] = (delta,)

    def set_chain(self, slot, next_slot, stream=None):
        """After the app of `slot`, apply the app of `next_slot` to the same row (-1 removes the link)."""
        self._check(self.lib.mix_set_chain(self.ctx, int(slot), int(next_slot), _stream(stream)))

    def apply_router(self, logits, T=None, stream=None):
        assert logits.dtype == torch.float32 and logits.is_cuda and logits.is_contiguous() and logits.dim() == 2
        T = logits.shape[0] if T is None else T
        self._check(self.lib.mix_apply_router(self.ctx, logits.data_ptr(), int(logits.shape[1]), int(T), _stream(stream)))

    @staticmethod
    def _edit_arrays(idx, val, mode):
        idx = np.ascontiguousarray(idx, dtype=np.int32)
        val = np.ascontiguousarray(val, dtype=np.float32)
        mode = np.ascontiguousarray(mode, dtype=np.uint8)
        assert len(idx) == len(val) == len(mode)
        return idx, val, mode

    def register_sae_app(self, slot, group, idx, val, mode, add_error, stream=None):
        idx, val, mode = self._edit_arrays(idx, val, mode)
        d = MixSaeApp(int(group), len(idx), idx.ctypes.data, val.ctypes.data, mode.ctypes.data, int(bool(add_error)))
        self._check(self.lib.mix_register_app(self.ctx, slot, MIX_SAE, C.byref(d), _stream(stream)))

    def unregister_app(self, slot, stream=None):
        self._check(self.lib.mix_unregister_app(self.ctx, slot, _stream(stream)))
        self._keep.pop(("a", slot), None)

    def set_gate(self, slot, scores, column=0, cmp=MIX_GATE_GE, threshold=0.0, stream=None):
        """Gate the app in `slot` on scores[t, column] (CUDA fp32 [T_max, stride]); scores=None removes it."""
        if scores is None:
            self._check(self.lib.mix_set_gate(self.ctx, slot, None, 1, 0, 0, 0.0, _stream(stream)))
            self._keep.pop(("gate", slot), None)
            return
        assert scores.dtype == torch.float32 and scores.dim() == 2
        self._check(self.lib.mix_set_gate(self.ctx, slot, _ptr(scores), int(scores.shape[1]), int(column), int(cmp),
                                          float(threshold), _stream(stream)))
        self._keep[("gate", slot)] = scores

    def update_steer_alpha(self, slot, alpha, stream=None):
        self._check(self.lib.mix_update_steer_alpha(self.ctx, slot, float(alpha), _stream(stream)))

    def update_sae_edits(self, slot, idx, val, mode, stream=None):
        idx, val, mode = self._edit_arrays(idx, val, mode)
        self._check(self.lib.mix_update_sae_edits(self.ctx, slot, len(idx), idx.ctypes.data, val.ctypes.data,
                                                  mode.ctypes.data, _stream(stream)))

    def set_slot_map(self, token_slot, T_live=None, stream=None):
        """token_slot: int32 torch tensor (CUDA, or CPU -- pinned for an async copy) or numpy array."""
        if isinstance(token_slot, np.ndarray):
            token_slot = np.ascontiguousarray(token_slot, dtype=np.int32)
            n = len(token_slot) if T_live is None else T_live
            self._check(self.lib.mix_set_slot_map(self.ctx, token_slot.ctypes.data, n, 0, _stream(stream)))
            return
        assert token_slot.dtype == torch.int32 and token_slot.is_contiguous()
        n = token_slot.numel() if T_live is None else T_live
        self._check(self.lib.mix_set_slot_map(self.ctx, token_slot.data_ptr(), n, int(token_slot.is_cuda),
                                              _stream(stream)))

    def set_request_map(self, token_req, req_slot, T_live=None, stream=None):
        if isinstance(token_req, np.ndarray):
            token_req = np.ascontiguousarray(token_req, dtype=np.int32)
            req_slot = np.ascontiguousarray(req_slot, dtype=np.int32)
            n = len(token_req) if T_live is None else T_live
            self._check(self.lib.mix_set_request_map(self.ctx, token_req.ctypes.data, n, req_slot.ctypes.data,
                                                     len(req_slot), 0, _stream(stream)))
            return
        n = token_req.numel() if T_live is None else T_live
        self._check(self.lib.mix_set_request_map(self.ctx, token_req.data_ptr(), n, req_slot.data_ptr(),
                                                 req_slot.numel(), int(token_req.is_cuda), _stream(stream)))

    def set_feature_out(self, topk_idx=None, topk_val=None, n_active=None):
        self._check(self.lib.mix_set_feature_out(self.ctx, _ptr(topk_idx), _ptr(topk_val), _ptr(n_active)))
        self._keep["fo"] = (topk_idx, topk_val, n_active)

    def apply(self, hidden, scores_out=None, T=None, stream=None):
        assert hidden.dtype == torch.bfloat16 and hidden.is_cuda and hidden.is_contiguous()
        T = hidden.shape[0] if T is None else T
        self._check(self.lib.mix_apply(self.ctx, hidden.data_ptr(), int(T), _ptr(scores_out), _stream(stream)))

    def apply_conditional(self, hidden, scores_out=None, T=None, stream=None):
        """As apply(), inside a stream capture only: the SAE chain becomes the body of a graph IF node."""
        assert hidden.dtype == torch.bfloat16 and hidden.is_cuda and hidden.is_contiguous()
        T = hidden.shape[0] if T is None else T
        self._check(self.lib.mix_apply_conditional(self.ctx, hidden.data_ptr(), int(T), _ptr(scores_out),
                                                   _stream(stream)))

    def get_status(self, stream=None) -> int:
        bits = C.c_uint(0)
        self._check(self.lib.mix_get_status(self.ctx, C.byref(bits), _stream(stream)))
        return int(bits.value)

    def launches_per_apply(self) -> int:
        return int(self.lib.mix_launches_per_apply(self.ctx))

    @property
    def STAGES(self):
        front = ["probe_steer"]
        if self.cfg.T_max > 2048 and self.cfg.C_max > 1 and not (self.cfg.flags & MIX_FLAG_SLOT_CHAINS):
            front.append("probe_multiclass")
            if self.cfg.n_groups_max == 0:
                front = ["probe_decide"] + front + ["probe_tc"]
        if self.cfg.n_groups_max == 0:
            return front
        tail = ["edit_only", "edit_only_delta"] if self.cfg.flags & MIX_FLAG_SAE_EDIT_ONLY else []
        if self.cfg.flags & MIX_FLAG_ENCODE_SIMT:
            return front + ["front", "encode", "tail"] + tail
        return front + ["front", "encode", "encode_pair", "tail", "encode_flagged", "tail_flagged"] + tail

    def set_stage_events(self, events=None):
        """events: list of launches_per_apply() + 1 torch.cuda.Event(enable_timing=True), or None."""
        if events is None:
            self._check(self.lib.mix_set_stage_events(self.ctx, None))
            self._keep.pop("ev", None)
            return
        for e in events:
            e.record()                       # torch creates the CUDA event lazily, on first record
        arr = (C.c_void_p * len(events))(*[e.cuda_event for e in events])
        self._check(self.lib.mix_set_stage_events(self.ctx, arr))
        self._keep["ev"] = events

    def bench_param_update(self, iters=2000, stream=None):
        """(us per iteration with a device-table write, us per iteration with a kernel-node parameter update)."""
        a, b = C.c_float(0), C.c_float(0)
        self._check(self.lib.mix_bench_param_update(self.ctx, int(iters), C.byref(a), C.byref(b), _stream(stream)))
        return float(a.value), float(b.value)

    def debug_phase_clocks(self):
        """32 nanosecond stamps of the front / tail kernels' phases (zeros unless MIX_PHASE_CLOCKS=1 at creation)."""
        out = (C.c_ulonglong * 32)()
        self._check(self.lib.mix_debug_phase_clocks(self.ctx, out))
        return [int(x) for x in out]

    def debug_workspace(self):
        pr, z, ld, n = C.c_void_p(), C.c_void_p(), C.c_longlong(), C.c_int()
        self._check(self.lib.mix_debug_workspace(self.ctx, C.byref(pr), C.byref(z), C.byref(ld), C.byref(n)))
        return pr.value, z.value, ld.value, n.value


STATIC_MAX_ROWS, STATIC_MAX_D_MODEL, STATIC_MAX_D_SAE, STATIC_MAX_K = 128, 4096, 8192, 128


def sae_apply_static(hidden, d_sae, act, k, W_enc, b_enc, W_dec, idx, val, mode, add_error, theta=None, b_dec=None,
                     topk_idx=None, topk_val=None, stream=None):
    """The SAE function on every row of `hidden` (CUDA bf16 [n_rows, d], in place) without any
    device allocation: for callers that may not call cudaMalloc (see mix_sae_apply_static in
    mix.h for who they are, the size limits, and why overlapping calls race).  Needs no Mix
    context.  Raises MixError with the library's message when a size exceeds the fixed limits."""
    lib = load_library()
    assert hidden.dtype == torch.bfloat16 and hidden.is_cuda and hidden.is_contiguous()
    idx, val, mode = Mix._edit_arrays(idx, val, mode)
    w = MixSaeWeights(int(d_sae), int(act), int(k), _ptr(W_enc), _ptr(b_enc), _ptr(theta), _ptr(W_dec), _ptr(b_dec), 0)
    a = MixSaeApp(0, len(idx), idx.ctypes.data, val.ctypes.data, mode.ctypes.data, int(bool(add_error)))
    err = C.create_string_buffer(256)
    rc = lib.mix_sae_apply_static(hidden.data_ptr(), int(hidden.shape[0]), int(hidden.shape[1]), C.byref(w),
                                  C.byref(a), _ptr(topk_idx), _ptr(topk_val), _stream(stream), err, 256)
    if rc != 0:
        raise MixError(rc, err.value.decode())
