"""Thin ctypes binding over libcca.so: argument marshalling only.

Every step of the block runs inside the library's CUDA kernels; torch is used here for device
memory and streams.  There is no CPU fallback: if the library cannot be loaded, or a call fails,
an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

from . import build as _build

_LIB = None


class CcaError(RuntimeError):
    pass


class cca_config(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("compression", C.c_int32), ("k_seq", C.c_int32), ("k_ch", C.c_int32),
                ("causal", C.c_int32), ("flags", C.c_uint32), ("rope_base", C.c_float)]


class cca_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_qk", "w_v1", "w_v2", "w_o", "conv0_w", "conv1_w", "temp")]


class cca_weight_grads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("d_w_qk", "d_w_v1", "d_w_v2", "d_w_o", "d_conv0_w", "d_conv1_w", "d_temp")]


class cca_layout(C.Structure):
    _fields_ = [("L_q", C.c_int64), ("L_k", C.c_int64), ("g", C.c_int64), ("total_padding", C.c_int64),
                ("v_shift_split", C.c_int64), ("q_to_kv_head", C.c_int64 * 64), ("conv_params", C.c_int64),
                ("params", C.c_int64), ("kv_cache_elems", C.c_int64), ("fwd_flops", C.c_int64),
                ("fwd_flops_causal", C.c_int64), ("decode_flops", C.c_int64),
                ("off_qk0", C.c_int64), ("off_q", C.c_int64), ("off_k", C.c_int64), ("off_v", C.c_int64),
                ("off_o", C.c_int64), ("off_lse", C.c_int64), ("off_rope", C.c_int64),
                ("saved_bytes", C.c_int64), ("total_bytes", C.c_int64), ("off_rnorm", C.c_int64)]


class cca_mla_dims(C.Structure):
    _fields_ = [("d_nope", C.c_int32), ("d_rope", C.c_int32), ("d_ckv", C.c_int32), ("d_cq", C.c_int32)]


MLA_WEIGHTS = ("w_dq", "w_dkv", "w_uq", "w_uqr", "w_uk", "w_uv", "w_kr", "w_o")


class cca_mla_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in MLA_WEIGHTS]


class cca_decode_state(C.Structure):
    _fields_ = [("k_cache", C.c_void_p), ("v_cache", C.c_void_p), ("qk0_hist", C.c_void_p), ("x_prev", C.c_void_p),
                ("pos", C.c_void_p), ("S_max", C.c_int64)]


# name -> (restype, argtypes); also the list of symbols the header declares
SYMBOLS = {
    "cca_init": (C.c_int, [C.POINTER(cca_config), C.c_int, C.POINTER(C.c_void_p)]),
    "cca_destroy": (C.c_int, [C.c_void_p]),
    "cca_describe": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.POINTER(cca_layout)]),
    "cca_workspace_size": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_int, C.POINTER(C.c_size_t)]),
    "cca_forward": (C.c_int, [C.c_void_p, C.POINTER(cca_weights), C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                              C.c_int64, C.c_int64, C.c_int, C.c_void_p]),
    "cca_backward": (C.c_int, [C.c_void_p, C.POINTER(cca_weights), C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                               C.c_void_p, C.POINTER(cca_weight_grads), C.c_int64, C.c_int64, C.c_void_p]),
    "cca_forward_host": (C.c_int, [C.c_void_p, C.POINTER(cca_weights), C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_size_t, C.c_int64, C.c_int64, C.c_void_p]),
    "cca_forward_chunk": (C.c_int, [C.c_void_p, C.POINTER(cca_weights), C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                    C.c_int64, C.c_int64, C.c_int64, C.c_void_p]),
    "cca_forward_static": (C.c_int, [C.c_void_p, C.POINTER(cca_weights), C.c_void_p, C.c_void_p, C.c_int64, C.c_int64,
                                     C.c_void_p]),
    "cca_attention_forward": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_int64, C.c_int64, C.c_void_p]),
    "cca_decode_workspace_size": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.POINTER(C.c_size_t)]),
    "cca_decode_step": (C.c_int, [C.c_void_p, C.POINTER(cca_weights), C.c_void_p, C.c_void_p, C.POINTER(cca_decode_state),
                                  C.c_int64, C.c_void_p, C.c_size_t, C.c_int64, C.c_void_p]),
    "cca_decode_state_from_prefill": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_int64, C.c_int64,
                                                C.POINTER(cca_decode_state), C.c_void_p]),
    "cca_mla_workspace_size": (C.c_int, [C.c_void_p, C.POINTER(cca_mla_dims), C.c_int64, C.c_int64, C.POINTER(C.c_size_t)]),
    "cca_mla_forward": (C.c_int, [C.c_void_p, C.POINTER(cca_mla_dims), C.POINTER(cca_mla_weights), C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.c_size_t, C.c_int64, C.c_int64, C.c_void_p]),
    "cca_set_impl": (C.c_int, [C.c_void_p, C.c_int]),
    "cca_set_attention_events": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "cca_set_stage_events": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.c_int]),
    "cca_launch_count": (C.c_int64, [C.c_void_p]),
    "cca_last_status": (C.c_int, [C.c_void_p, C.POINTER(C.c_int)]),
    "cca_set_wait_limit": (C.c_int, [C.c_void_p, C.c_int64]),
    "cca_wait_selftest": (C.c_int, [C.c_void_p, C.c_void_p]),
    "cca_last_cuda_error": (C.c_int, [C.c_void_p]),
    "cca_status_string": (C.c_char_p, [C.c_int]),
}


def lib_path() -> str:
    return _build.LIB


def load_library(build_if_missing: bool = True) -> C.CDLL:
    """Load libcca.so (building it first if it is missing or stale).  Raises if that fails."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = _build.build() if build_if_missing else _build.LIB
    if not os.path.exists(path):
        raise CcaError(f"{path} is missing: build the CUDA library first (python -m paper_2510_04476_b200.build)")
    lib = C.CDLL(path)
    for name, (res, args) in SYMBOLS.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _LIB = lib
    return lib


def _check(lib, code: int, handle=None, what: str = ""):
    if code != 0:
        msg = lib.cca_status_string(code).decode()
        extra = ""
        if handle is not None and code == 5:
            extra = f" (cudaError {lib.cca_last_cuda_error(handle)})"
        raise CcaError(f"{what}: {msg}{extra}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def stack_down_projection(w: Dict[str, torch.Tensor]) -> Dict[str, torch.Tensor]:
    """The same parameters with w_qk, w_v1, w_v2 as views of one [L + L_k, E] device tensor, the layout the library
    reads in place (see cca_weights in the header).  Memory placement only."""
    out = dict(w)
    allw = torch.cat([w["w_qk"], w["w_v1"], w["w_v2"]], dim=0).contiguous()
    n0, n1 = w["w_qk"].shape[0], w["w_v1"].shape[0]
    out["w_qk"], out["w_v1"], out["w_v2"] = allw[:n0], allw[n0:n0 + n1], allw[n0 + n1:]
    return out


class CCA:
    """One configured block on one device.  Methods mirror the C entry points."""

    def __init__(self, d_model, n_q_heads, n_kv_heads, head_dim, k_seq=2, k_ch=2, causal=1, flags=63,
                 rope_base=10000.0, device=0, compression=None):
        self.lib = load_library()
        if compression is None:
            compression = d_model // max(1, n_q_heads * head_dim)
        self.cfg = cca_config(d_model, n_q_heads, n_kv_heads, head_dim, compression, k_seq, k_ch, causal, flags,
                              rope_base)
        self.device = torch.device("cuda", device)
        self.handle = C.c_void_p()
        _check(self.lib, self.lib.cca_init(C.byref(self.cfg), device, C.byref(self.handle)), None, "cca_init")

    @classmethod
    def from_shape(cls, sh, device=0) -> "CCA":
        return cls(sh.d_model, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.k_seq, sh.k_ch, sh.causal, sh.flags,
                   sh.rope_base, device)

    def close(self):
        if getattr(self, "handle", None) is not None and self.handle.value:
            self.lib.cca_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- metadata -------------------------------------------------------------------------
    def describe(self, B: int, S: int) -> Dict[str, object]:
        lay = cca_layout()
        _check(self.lib, self.lib.cca_describe(self.handle, B, S, C.byref(lay)), self.handle, "cca_describe")
        out = {}
        for name, _ in cca_layout._fields_:
            val = getattr(lay, name)
            out[name] = list(val) if name == "q_to_kv_head" else int(val)
        return out

    def workspace_size(self, B: int, S: int, need_backward: bool = True) -> int:
        n = C.c_size_t()
        _check(self.lib, self.lib.cca_workspace_size(self.handle, B, S, int(need_backward), C.byref(n)), self.handle,
               "cca_workspace_size")
        return int(n.value)

    def alloc_workspace(self, B: int, S: int, need_backward: bool = True, extra: int = 0) -> torch.Tensor:
        return torch.empty(self.workspace_size(B, S, need_backward) + extra + 256, dtype=torch.uint8,
                           device=self.device)

    @staticmethod
    def _ws_ptr(ws: torch.Tensor):
        p = ws.data_ptr()
        a = (p + 255) // 256 * 256
        return C.c_void_p(a), ws.numel() - (a - p)

    def set_impl(self, impl: int) -> int:
        return self.lib.cca_set_impl(self.handle, impl)

    def set_attention_events(self, begin: Optional[torch.cuda.Event], end: Optional[torch.cuda.Event]):
        """Events (created with enable_timing=True) recorded around the attention kernel; None clears."""
        for e in (begin, end):
            if e is not None and e.cuda_event == 0:
                e.record(torch.cuda.current_stream(self.device))      # forces creation of the handle
        b = C.c_void_p(begin.cuda_event) if begin is not None else None
        e = C.c_void_p(end.cuda_event) if end is not None else None
        _check(self.lib, self.lib.cca_set_attention_events(self.handle, b, e), self.handle, "set_attention_events")

    STAGE_EVENTS = ["fwd_begin", "fwd_proj", "fwd_transform", "fwd_attn", "fwd_end", "bwd_begin", "bwd_do", "bwd_dwo",
                    "bwd_delta", "bwd_attn", "bwd_norm", "bwd_conv2", "bwd_conv1", "bwd_pack", "bwd_dw", "bwd_end"]

    def set_stage_events(self, events):
        """cca_set_stage_events: a list of len(STAGE_EVENTS) torch.cuda.Event(enable_timing=True), or None to clear."""
        if events is None:
            _check(self.lib, self.lib.cca_set_stage_events(self.handle, None, 0), self.handle, "cca_set_stage_events")
            return
        assert len(events) == len(self.STAGE_EVENTS)
        for e in events:
            if e.cuda_event == 0:
                e.record(torch.cuda.current_stream(self.device))      # forces creation of the handle
        arr = (C.c_void_p * len(events))(*[e.cuda_event for e in events])
        _check(self.lib, self.lib.cca_set_stage_events(self.handle, arr, len(events)), self.handle, "cca_set_stage_events")

    def launch_count(self) -> int:
        return int(self.lib.cca_launch_count(self.handle))

    def last_status(self) -> int:
        s = C.c_int()
        self.lib.cca_last_status(self.handle, C.byref(s))
        return int(s.value)

    # ---- compute --------------------------------------------------------------------------
    def _weights(self, w: Dict[str, torch.Tensor]) -> cca_weights:
        cw = cca_weights()
        for n in ("w_qk", "w_v1", "w_v2", "w_o", "conv0_w", "conv1_w", "temp"):
            t = w.get(n)
            if t is not None:
                assert t.is_cuda and t.is_contiguous(), n
                assert t.dtype == (torch.float32 if n == "temp" else torch.bfloat16), n
            setattr(cw, n, t.data_ptr() if t is not None else None)
        return cw

    def forward(self, w, x: torch.Tensor, workspace: torch.Tensor, out: Optional[torch.Tensor] = None,
                save_for_backward: Optional[bool] = None):
        """cca_forward.  save_for_backward=None: keep the activations for a backward exactly when the workspace was
        sized for one (alloc_workspace(..., need_backward=True))."""
        B, S, E = x.shape
        assert x.is_cuda and x.is_contiguous() and x.dtype == torch.bfloat16
        if out is None:
            out = torch.empty_like(x)
        cw = self._weights(w)
        wp, wn = self._ws_ptr(workspace)
        if save_for_backward is None:
            save_for_backward = wn >= self.workspace_size(B, S, True)
        st = C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)
        _check(self.lib, self.lib.cca_forward(self.handle, C.byref(cw), _ptr(x), _ptr(out), wp, wn, B, S,
                                              int(bool(save_for_backward)), st), self.handle, "cca_forward")
        return out

    def set_wait_limit(self, sm_cycles: int):
        _check(self.lib, self.lib.cca_set_wait_limit(self.handle, int(sm_cycles)), self.handle, "cca_set_wait_limit")

    def wait_selftest(self):
        st = C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)
        _check(self.lib, self.lib.cca_wait_selftest(self.handle, st), self.handle, "cca_wait_selftest")

    def last_status_code(self):
        """(return code of cca_last_status, device status word)."""
        s = C.c_int()
        rc = self.lib.cca_last_status(self.handle, C.byref(s))
        return int(rc), int(s.value)

    def forward_chunk(self, w, x_chunk: torch.Tensor, workspace: torch.Tensor, S_total: int, t_begin: int,
                      out: Optional[torch.Tensor] = None):
        """cca_forward_chunk: tokens [t_begin, t_begin + len(x_chunk)) of one causal sequence of S_total tokens."""
        n, E = x_chunk.shape
        assert x_chunk.is_cuda and x_chunk.is_contiguous() and x_chunk.dtype == torch.bfloat16
        if out is None:
            out = torch.empty_like(x_chunk)
        cw = self._weights(w)
        wp, wn = self._ws_ptr(workspace)
        st = C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)
        _check(self.lib, self.lib.cca_forward_chunk(self.handle, C.byref(cw), _ptr(x_chunk), _ptr(out), wp, wn, S_total,
                                                    t_begin, t_begin + n, st), self.handle, "cca_forward_chunk")
        return out

    def forward_host(self, w, x_host: torch.Tensor, out_host: torch.Tensor, workspace: torch.Tensor):
        B, S, E = x_host.shape
        assert not x_host.is_cuda and not out_host.is_cuda
        cw = self._weights(w)
        wp, wn = self._ws_ptr(workspace)
        st = C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)
        _check(self.lib, self.lib.cca_forward_host(self.handle, C.byref(cw), _ptr(x_host), _ptr(out_host), wp, wn,
                                                   B, S, st), self.handle, "cca_forward_host")
        return out_host

    def forward_static(self, w, x: torch.Tensor, out: torch.Tensor):
        """cca_forward_static: the forward with the library's built-in scratch; `out` is caller-provided and
        nothing is allocated on the way (not here either)."""
        B, S, E = x.shape
        assert x.is_cuda and x.is_contiguous() and x.dtype == torch.bfloat16
        assert out.is_cuda and out.is_contiguous() and out.dtype == torch.bfloat16 and out.shape == x.shape
        cw = self._weights(w)
        st = C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)
        _check(self.lib, self.lib.cca_forward_static(self.handle, C.byref(cw), _ptr(x), _ptr(out), B, S, st),
               self.handle, "cca_forward_static")
        return out

    # ---- decode ---------------------------------------------------------------------------
    def new_decode_state(self, B: int, S_max: int) -> Dict[str, torch.Tensor]:
        """Caller-owned tensors of cca_decode_state for B empty sequences (device memory only, no arithmetic)."""
        c = self.cfg
        Lk = c.n_kv_heads * c.head_dim
        L = c.n_q_heads * c.head_dim + Lk
        pad = c.k_seq + c.k_ch - 2
        dev = self.device
        return {"k_cache": torch.zeros(B, S_max, Lk, dtype=torch.bfloat16, device=dev),
                "v_cache": torch.zeros(B, S_max, Lk, dtype=torch.bfloat16, device=dev),
                "qk0_hist": torch.zeros(B, max(pad, 1), L, dtype=torch.float32, device=dev)[:, :pad].contiguous(),
                "x_prev": torch.zeros(B, c.d_model, dtype=torch.bfloat16, device=dev),
                "pos": torch.zeros(B, dtype=torch.int32, device=dev)}

    @staticmethod
    def _decode_state(state: Dict[str, torch.Tensor]) -> cca_decode_state:
        s = cca_decode_state()
        for n in ("k_cache", "v_cache", "qk0_hist", "x_prev", "pos"):
            t = state[n]
            assert t.is_cuda and t.is_contiguous(), n
            setattr(s, n, t.data_ptr() if t.numel() else None)
        assert state["pos"].dtype == torch.int32
        s.S_max = state["k_cache"].shape[1]
        return s

    def decode_workspace_size(self, B: int, max_len: int) -> int:
        n = C.c_size_t()
        _check(self.lib, self.lib.cca_decode_workspace_size(self.handle, B, max_len, C.byref(n)), self.handle,
               "cca_decode_workspace_size")
        return int(n.value)

    def alloc_decode_workspace(self, B: int, max_len: int) -> torch.Tensor:
        return torch.empty(self.decode_workspace_size(B, max_len) + 256, dtype=torch.uint8, device=self.device)

    def decode_step(self, w, x: torch.Tensor, state: Dict[str, torch.Tensor], max_len: int, workspace: torch.Tensor,
                    out: Optional[torch.Tensor] = None):
        """cca_decode_step: x [B,E] -> out [B,E]; the state tensors are updated in place except `pos`."""
        B, E = x.shape
        assert x.is_cuda and x.is_contiguous() and x.dtype == torch.bfloat16
        if out is None:
            out = torch.empty_like(x)
        cw = self._weights(w)
        ds = self._decode_state(state)
        wp, wn = self._ws_ptr(workspace)
        st = C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)
        _check(self.lib, self.lib.cca_decode_step(self.handle, C.byref(cw), _ptr(x), _ptr(out), C.byref(ds), max_len,
                                                  wp, wn, B, st), self.handle, "cca_decode_step")
        return out

    def decode_state_from_prefill(self, x: torch.Tensor, workspace: torch.Tensor, state: Dict[str, torch.Tensor]):
        B, S, E = x.shape
        ds = self._decode_state(state)
        wp, wn = self._ws_ptr(workspace)
        st = C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)
        _check(self.lib, self.lib.cca_decode_state_from_prefill(self.handle, _ptr(x), wp, wn, B, S, C.byref(ds), st),
               self.handle, "cca_decode_state_from_prefill")

    def backward(self, w, x: torch.Tensor, d_out: torch.Tensor, workspace: torch.Tensor, separate_grads: bool = False):
        """Returns (d_x bf16, dict of fp32 parameter gradients).  separate_grads: give every gradient a buffer of
        its own instead of one block for the three down-projection gradients."""
        B, S, E = x.shape
        assert d_out.is_cuda and d_out.is_contiguous() and d_out.dtype == torch.bfloat16
        d_x = torch.empty_like(x)
        grads = {}
        cg = cca_weight_grads()
        # the three down-projection gradients as one block (the library then writes them with one contraction)
        n0, n1, n2 = w["w_qk"].shape[0], w["w_v1"].shape[0], w["w_v2"].shape[0]
        if separate_grads:
            for n in ("w_qk", "w_v1", "w_v2"):
                grads["d_" + n] = torch.empty((w[n].shape[0] + 3, E), dtype=torch.float32, device=self.device)[:w[n].shape[0]]
        else:
            d_all = torch.empty((n0 + n1 + n2, E), dtype=torch.float32, device=self.device)
            grads["d_w_qk"], grads["d_w_v1"], grads["d_w_v2"] = d_all[:n0], d_all[n0:n0 + n1], d_all[n0 + n1:]
        c = self.cfg
        L = (c.n_q_heads + c.n_kv_heads) * c.head_dim
        shapes = {"w_o": (E, c.n_q_heads * c.head_dim), "conv0_w": (L, c.k_seq), "conv1_w": (L, c.head_dim, c.k_ch),
                  "temp": (c.n_kv_heads,)}
        for n, shp in shapes.items():
            grads["d_" + n] = torch.empty(shp, dtype=torch.float32, device=self.device)
        for n in ("w_qk", "w_v1", "w_v2", "w_o", "conv0_w", "conv1_w", "temp"):
            setattr(cg, "d_" + n, grads["d_" + n].data_ptr())
        cw = self._weights(w)
        wp, wn = self._ws_ptr(workspace)
        st = C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)
        _check(self.lib, self.lib.cca_backward(self.handle, C.byref(cw), _ptr(x), _ptr(d_out), wp, wn, _ptr(d_x),
                                               C.byref(cg), B, S, st), self.handle, "cca_backward")
        return d_x, grads

    def mla_forward(self, dims, w, x: torch.Tensor, out: Optional[torch.Tensor] = None):
        """cca_mla_forward.  dims = (d_nope, d_rope, d_ckv, d_cq); w: dict of the eight bf16 weights.  Returns (out, workspace)."""
        B, S, E = x.shape
        md = cca_mla_dims(*dims)
        n = C.c_size_t()
        _check(self.lib, self.lib.cca_mla_workspace_size(self.handle, C.byref(md), B, S, C.byref(n)), self.handle,
               "cca_mla_workspace_size")
        key = (B, S, tuple(dims))
        if getattr(self, "_mla_ws_key", None) != key:              # the workspace is kept between calls of one shape
            self._mla_ws = torch.empty(int(n.value) + 256, dtype=torch.uint8, device=self.device)
            self._mla_ws_key = key
        ws = self._mla_ws
        if out is None:
            out = torch.empty_like(x)
        mw = cca_mla_weights()
        for name in MLA_WEIGHTS:
            t = w[name]
            assert t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16, name
            setattr(mw, name, t.data_ptr())
        wp, wn = self._ws_ptr(ws)
        st = C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)
        _check(self.lib, self.lib.cca_mla_forward(self.handle, C.byref(md), C.byref(mw), _ptr(x), _ptr(out), wp, wn, B, S, st),
               self.handle, "cca_mla_forward")
        return out, ws

    def attention_forward(self, q, k, v, o=None, lse=None):
        B, S, hq, dh = q.shape
        if o is None:
            o = torch.empty_like(q)
        if lse is None:
            lse = torch.empty(B, hq, S, dtype=torch.float32, device=q.device)
        st = C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)
        _check(self.lib, self.lib.cca_attention_forward(self.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse),
                                                        B, S, st), self.handle, "cca_attention_forward")
        return o, lse

    def saved(self, workspace: torch.Tensor, B: int, S: int) -> Dict[str, torch.Tensor]:
        """Views of the activations cca_forward left in the workspace (for tests)."""
        lay = self.describe(B, S)
        wp, _ = self._ws_ptr(workspace)
        base = wp.value - workspace.data_ptr()
        cfg = self.cfg
        hq, hk, dh = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
        Lq, Lk = hq * dh, hk * dh

        def view(off, shape, dtype):
            n = 1
            for s in shape:
                n *= s
            nbytes = n * torch.empty((), dtype=dtype).element_size()
            return workspace[base + off: base + off + nbytes].view(dtype).view(*shape)

        return {
            "qk0": view(lay["off_qk0"], (B, S, Lq + Lk), torch.float32),
            "q": view(lay["off_q"], (B, S, hq, dh), torch.bfloat16),
            "k": view(lay["off_k"], (B, S, hk, dh), torch.bfloat16),
            "v": view(lay["off_v"], (B, S, hk, dh), torch.bfloat16),
            "o": view(lay["off_o"], (B, S, hq, dh), torch.bfloat16),
            "lse": view(lay["off_lse"], (B, hq, S), torch.float32),
        }
