"""ctypes binding of libmustdrop.so: argument marshalling only.

Every step of the filter runs in the CUDA library; nothing here computes.  The functions
carry the names of the C entry points (see include/mustdrop.h).  Device buffers are passed
as torch CUDA tensors (or raw integer device pointers); torch is used for memory and
streams only.  If the shared library is missing the import of any entry point raises:
there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
from typing import Optional, Tuple

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmustdrop.so")

MUSTDROP_OK = 0
MUSTDROP_ERR_INVALID_ARG = 1
MUSTDROP_ERR_UNSUPPORTED = 2
MUSTDROP_ERR_BUDGET = 3
MUSTDROP_ERR_WORKSPACE = 4
MUSTDROP_ERR_CUDA = 5
MUSTDROP_ERR_TIMEOUT = 6
MUSTDROP_ERR_BAD_KEY_INDEX = 7
MUSTDROP_ERR_SCRATCH_LIMIT = 8

MUSTDROP_MODE_BUDGET, MUSTDROP_MODE_THRESHOLD = 0, 1
MUSTDROP_CRIT_DUAL, MUSTDROP_CRIT_GLOBAL_ONLY, MUSTDROP_CRIT_INDIVIDUAL_ONLY = 0, 1, 2

EXPORTS = (
    "mustdrop_filter_plan", "mustdrop_plan_destroy", "mustdrop_score", "mustdrop_select",
    "mustdrop_compact", "mustdrop_device_status", "mustdrop_status_string",
    "mustdrop_last_cuda_error", "mustdrop_plan_score_variant", "mustdrop_score_static",
    "mustdrop_score_static_max_rows", "mustdrop_filter", "mustdrop_plan_filter_launches",
    "mustdrop_filter_layer", "mustdrop_cache_compact", "mustdrop_spatial_merge", "mustdrop_key_set",
    "mustdrop_plan_describe",
)


class mustdrop_config_t(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("n_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("hidden", ctypes.c_int32), ("seq_len", ctypes.c_int32), ("vis_start", ctypes.c_int32),
        ("n_vis", ctypes.c_int32), ("txt_start", ctypes.c_int32), ("n_txt", ctypes.c_int32),
        ("causal", ctypes.c_int32), ("scale", ctypes.c_float), ("mode", ctypes.c_int32),
        ("criteria", ctypes.c_int32), ("budget", ctypes.c_int32), ("gamma", ctypes.c_float),
        ("alpha", ctypes.c_float), ("key_max", ctypes.c_int32), ("flags", ctypes.c_int32),
        ("k_stride_b", ctypes.c_int64), ("k_stride_h", ctypes.c_int64), ("k_stride_l", ctypes.c_int64),
        ("v_stride_b", ctypes.c_int64), ("v_stride_h", ctypes.c_int64), ("v_stride_l", ctypes.c_int64),
        ("hid_stride_b", ctypes.c_int64), ("hid_stride_l", ctypes.c_int64),
        ("debug_score_variant", ctypes.c_int32), ("debug_cluster", ctypes.c_int32),
        ("debug_filter_staged", ctypes.c_int32), ("debug_wait_cycles", ctypes.c_int32),
    ]


MUSTDROP_FLAG_REBUILD_SEQUENCE = 1
MUSTDROP_FLAG_PER_HEAD_MAX = 2
MUSTDROP_FLAG_INPUTS_READY = 4

MUSTDROP_DEBUG_VARIANT_AUTO, MUSTDROP_DEBUG_VARIANT_TWO_PASS = 0, 1
MUSTDROP_DEBUG_VARIANT_FUSED, MUSTDROP_DEBUG_VARIANT_ROW_SPLIT = 2, 3
MUSTDROP_DEBUG_VARIANT_GRID = 4


class mustdrop_layer_io_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in (
        "q_text", "k", "v", "hidden", "key_idx", "key_cnt", "vis_cnt", "orig_idx", "g_out", "i_out", "s_out",
        "kept_idx", "kept_cnt", "orig_out", "key_idx_out", "key_cnt_out", "hidden_out", "k_out", "v_out")]


class mustdrop_cache_config_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "n_layers", "batch", "n_heads", "head_dim", "rows_in", "vis_start", "n_tail", "ids_max", "cap")]


class MustDropError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().mustdrop_status_string(status).decode()
        if status == MUSTDROP_ERR_CUDA:
            msg += " (cudaError %d)" % lib().mustdrop_last_cuda_error()
        super().__init__("%s: %s" % (where, msg))


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libmustdrop.so is missing (%s): build it with `python -m paper_2411_10803_b200.build`; "
                "there is no CPU fallback" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, i32p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32)
        L.mustdrop_filter_plan.argtypes = [ctypes.POINTER(mustdrop_config_t), ctypes.POINTER(vp),
                                           ctypes.POINTER(ctypes.c_size_t)]
        L.mustdrop_plan_destroy.argtypes = [vp]
        L.mustdrop_score.argtypes = [vp] * 7
        L.mustdrop_select.argtypes = [vp] * 10
        L.mustdrop_score_static.argtypes = [vp] * 6
        L.mustdrop_score_static.restype = ctypes.c_int
        L.mustdrop_score_static_max_rows.restype = ctypes.c_size_t
        L.mustdrop_compact.argtypes = [vp] * 11
        L.mustdrop_filter.argtypes = [vp] * 17
        L.mustdrop_filter_layer.argtypes = [vp, ctypes.POINTER(mustdrop_layer_io_t), vp, vp]
        L.mustdrop_cache_compact.argtypes = [ctypes.POINTER(mustdrop_cache_config_t)] + [vp] * 10
        L.mustdrop_cache_compact.restype = ctypes.c_int
        i32, f32 = ctypes.c_int32, ctypes.c_float
        L.mustdrop_spatial_merge.argtypes = [i32, i32, i32, i32, f32, vp, vp, vp, vp, vp, vp]
        L.mustdrop_spatial_merge.restype = ctypes.c_int
        L.mustdrop_key_set.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        L.mustdrop_key_set.restype = ctypes.c_int
        L.mustdrop_plan_filter_launches.argtypes = [vp]
        L.mustdrop_plan_filter_launches.restype = ctypes.c_int32
        L.mustdrop_device_status.argtypes = [vp, vp, vp, i32p, i32p]
        L.mustdrop_status_string.argtypes = [ctypes.c_int]
        L.mustdrop_status_string.restype = ctypes.c_char_p
        L.mustdrop_last_cuda_error.restype = ctypes.c_int32
        L.mustdrop_plan_score_variant.argtypes = [vp]
        L.mustdrop_plan_score_variant.restype = ctypes.c_char_p
        for n in ("mustdrop_filter_plan", "mustdrop_plan_destroy", "mustdrop_score", "mustdrop_select",
                  "mustdrop_compact", "mustdrop_filter", "mustdrop_filter_layer", "mustdrop_device_status"):
            getattr(L, n).restype = ctypes.c_int
        _lib = L
    return _lib


def _ptr(x) -> Optional[int]:
    """Device pointer of a torch tensor, an int, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


@dataclasses.dataclass
class Config:
    batch: int
    n_heads: int
    hidden: int
    seq_len: int
    vis_start: int
    n_vis: int
    txt_start: int
    n_txt: int
    head_dim: int = 128
    causal: int = 1
    scale: float = 0.0
    mode: int = MUSTDROP_MODE_BUDGET
    criteria: int = MUSTDROP_CRIT_DUAL
    budget: int = 0
    gamma: float = 0.0
    alpha: float = 0.0
    key_max: int = 0
    flags: int = 0
    k_stride_b: int = 0
    k_stride_h: int = 0
    k_stride_l: int = 0
    v_stride_b: int = 0
    v_stride_h: int = 0
    v_stride_l: int = 0
    hid_stride_b: int = 0
    hid_stride_l: int = 0
    debug_score_variant: int = 0
    debug_cluster: int = 0
    debug_filter_staged: int = 0
    debug_wait_cycles: int = 0

    def to_c(self) -> mustdrop_config_t:
        c = mustdrop_config_t()
        for f, _ in mustdrop_config_t._fields_:
            setattr(c, f, getattr(self, f))
        return c

    @property
    def cap(self) -> int:
        return self.budget if self.mode == MUSTDROP_MODE_BUDGET else self.n_vis

    @property
    def out_rows(self) -> int:
        """Rows per request (and head) of the compacted outputs."""
        if self.flags & MUSTDROP_FLAG_REBUILD_SEQUENCE:
            return self.vis_start + self.cap + self.n_txt
        return self.cap


def mustdrop_filter_plan(config: Config) -> Tuple[int, int, int]:
    """-> (status, plan handle, workspace bytes)."""
    c = config.to_c()
    plan = ctypes.c_void_p()
    ws = ctypes.c_size_t()
    st = lib().mustdrop_filter_plan(ctypes.byref(c), ctypes.byref(plan), ctypes.byref(ws))
    return st, plan.value or 0, ws.value


def mustdrop_plan_destroy(plan: int) -> int:
    return lib().mustdrop_plan_destroy(plan)


def mustdrop_score(plan, q_text, k, g_out, i_out, workspace, stream=None) -> int:
    return lib().mustdrop_score(plan, _ptr(q_text), _ptr(k), _ptr(g_out), _ptr(i_out), _ptr(workspace),
                                _stream(stream))


def mustdrop_score_static(plan, q_text, k, g_out, i_out, stream=None) -> int:
    """mustdrop_score without a workspace, for callers that may not allocate device memory: the
    scratch lives in a fixed array inside the library.  Calls that overlap on the GPU race on it."""
    return lib().mustdrop_score_static(plan, _ptr(q_text), _ptr(k), _ptr(g_out), _ptr(i_out), _stream(stream))


def mustdrop_score_static_max_rows() -> int:
    return lib().mustdrop_score_static_max_rows()


def mustdrop_select(plan, g, i, key_idx, key_cnt, kept_idx, kept_cnt, s_out, workspace, stream=None) -> int:
    return lib().mustdrop_select(plan, _ptr(g), _ptr(i), _ptr(key_idx), _ptr(key_cnt), _ptr(kept_idx),
                                 _ptr(kept_cnt), _ptr(s_out), _ptr(workspace), _stream(stream))


def mustdrop_compact(plan, kept_idx, kept_cnt, hidden, k, v, hidden_out, k_out, v_out, workspace,
                     stream=None) -> int:
    return lib().mustdrop_compact(plan, _ptr(kept_idx), _ptr(kept_cnt), _ptr(hidden), _ptr(k), _ptr(v),
                                  _ptr(hidden_out), _ptr(k_out), _ptr(v_out), _ptr(workspace), _stream(stream))


def mustdrop_filter(plan, q_text, k, v, hidden, key_idx, key_cnt, g_out, i_out, s_out, kept_idx, kept_cnt,
                    hidden_out, k_out, v_out, workspace, stream=None) -> int:
    return lib().mustdrop_filter(plan, _ptr(q_text), _ptr(k), _ptr(v), _ptr(hidden), _ptr(key_idx), _ptr(key_cnt),
                                 _ptr(g_out), _ptr(i_out), _ptr(s_out), _ptr(kept_idx), _ptr(kept_cnt),
                                 _ptr(hidden_out), _ptr(k_out), _ptr(v_out), _ptr(workspace), _stream(stream))


def mustdrop_filter_layer(plan, workspace, stream=None, **tensors) -> int:
    """Keyword arguments are the fields of mustdrop_layer_io_t (torch tensors, ints or None)."""
    io = mustdrop_layer_io_t()
    names = {n for n, _ in mustdrop_layer_io_t._fields_}
    for n, t in tensors.items():
        if n not in names:
            raise TypeError("mustdrop_layer_io_t has no field %r" % n)
        setattr(io, n, _ptr(t))
    return lib().mustdrop_filter_layer(plan, ctypes.byref(io), _ptr(workspace), _stream(stream))


def mustdrop_cache_compact(k_cache, v_cache, layer_ids, layer_cnt, s_few, s_few_cnt, k_out, v_out, workspace=None,
                           stream=None, **sizes) -> int:
    """sizes: the fields of mustdrop_cache_config_t (head_dim defaults to 128)."""
    c = mustdrop_cache_config_t()
    c.head_dim = 128
    for n, val in sizes.items():
        setattr(c, n, int(val))
    return lib().mustdrop_cache_compact(ctypes.byref(c), _ptr(k_cache), _ptr(v_cache), _ptr(layer_ids),
                                        _ptr(layer_cnt), _ptr(s_few), _ptr(s_few_cnt), _ptr(k_out), _ptr(v_out),
                                        _ptr(workspace), _stream(stream))


def mustdrop_spatial_merge(batch, grid, window, channels, tau, tokens, merged, slots, merged_cnt, window_sim=None,
                           stream=None) -> int:
    return lib().mustdrop_spatial_merge(batch, grid, window, channels, tau, _ptr(tokens), _ptr(merged), _ptr(slots),
                                        _ptr(merged_cnt), _ptr(window_sim), _stream(stream))


def mustdrop_key_set(batch, n_heads, head_dim, n_tokens, key_max, q_cls, k, a_cls, mu_out, key_idx, key_cnt,
                     stream=None) -> int:
    return lib().mustdrop_key_set(batch, n_heads, head_dim, n_tokens, key_max, _ptr(q_cls), _ptr(k), _ptr(a_cls),
                                  _ptr(mu_out), _ptr(key_idx), _ptr(key_cnt), _stream(stream))


def mustdrop_plan_describe(plan) -> str:
    buf = ctypes.create_string_buffer(256)
    L = lib()
    L.mustdrop_plan_describe.argtypes = [ctypes.c_void_p, ctypes.c_char_p, ctypes.c_size_t]
    L.mustdrop_plan_describe.restype = ctypes.c_int32
    L.mustdrop_plan_describe(plan, buf, 256)
    return buf.value.decode()


def mustdrop_plan_filter_launches(plan) -> int:
    return lib().mustdrop_plan_filter_launches(plan)


def mustdrop_device_status(plan, workspace, stream=None) -> Tuple[int, int, int]:
    """-> (status of the call, device code, detail)."""
    code, detail = ctypes.c_int32(0), ctypes.c_int32(0)
    st = lib().mustdrop_device_status(plan, _ptr(workspace), _stream(stream), ctypes.byref(code),
                                      ctypes.byref(detail))
    return st, code.value, detail.value


def mustdrop_status_string(status: int) -> str:
    return lib().mustdrop_status_string(status).decode()


def mustdrop_plan_score_variant(plan) -> str:
    return lib().mustdrop_plan_score_variant(plan).decode()


class Filter:
    """Convenience owner of a plan, its workspace and the output buffers (torch CUDA tensors).

    All arithmetic happens in the library calls; this class only allocates and forwards.
    """

    def __init__(self, config: Config, device="cuda"):
        import torch
        self.config = config
        st, self.plan, self.ws_bytes = mustdrop_filter_plan(config)
        if st != MUSTDROP_OK:
            raise MustDropError(st, "mustdrop_filter_plan")
        B, M, H, cap = config.batch, config.n_vis, config.n_heads, config.cap
        rows = config.out_rows
        self.device = torch.device(device)
        self.workspace = torch.zeros(self.ws_bytes, dtype=torch.uint8, device=self.device)
        self.g = torch.empty((B, M), dtype=torch.float32, device=self.device)
        self.i = torch.empty((B, M), dtype=torch.float32, device=self.device)
        self.s = torch.empty((B, M), dtype=torch.float32, device=self.device)
        self.kept_idx = torch.full((B, cap), -1, dtype=torch.int32, device=self.device)
        self.kept_cnt = torch.zeros((B,), dtype=torch.int32, device=self.device)
        self.hidden_out = torch.zeros((B, rows, config.hidden), dtype=torch.bfloat16, device=self.device)
        self.k_out = torch.zeros((B, H, rows, config.head_dim), dtype=torch.bfloat16, device=self.device)
        self.v_out = torch.zeros((B, H, rows, config.head_dim), dtype=torch.bfloat16, device=self.device)
        self.orig_out = torch.full((B, cap), -1, dtype=torch.int32, device=self.device)
        self.key_idx_out = torch.full((B, max(config.key_max, 1)), -1, dtype=torch.int32, device=self.device)
        self.key_cnt_out = torch.zeros((B,), dtype=torch.int32, device=self.device)

    def close(self):
        if getattr(self, "plan", 0):
            mustdrop_plan_destroy(self.plan)
            self.plan = 0

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def _check(st, where):
        if st != MUSTDROP_OK:
            raise MustDropError(st, where)

    def score(self, q_text, k, stream=None):
        self._check(mustdrop_score(self.plan, q_text, k, self.g, self.i, self.workspace, stream), "mustdrop_score")
        return self.g, self.i

    def select(self, key_idx=None, key_cnt=None, g=None, i=None, stream=None, want_s=True):
        self._check(mustdrop_select(self.plan, self.g if g is None else g, self.i if i is None else i,
                                    key_idx, key_cnt, self.kept_idx, self.kept_cnt,
                                    self.s if want_s else None, self.workspace, stream), "mustdrop_select")
        return self.kept_idx, self.kept_cnt

    def compact(self, hidden, k, v, kept_idx=None, kept_cnt=None, stream=None):
        self._check(mustdrop_compact(self.plan, self.kept_idx if kept_idx is None else kept_idx,
                                     self.kept_cnt if kept_cnt is None else kept_cnt, hidden, k, v,
                                     self.hidden_out if hidden is not None else None,
                                     self.k_out if k is not None else None,
                                     self.v_out if v is not None else None, self.workspace, stream),
                    "mustdrop_compact")
        return self.hidden_out, self.k_out, self.v_out

    def run(self, q_text, k, v, hidden, key_idx=None, key_cnt=None, stream=None, want_s=False):
        """score -> select -> compact on one stream, no host synchronisation."""
        self.score(q_text, k, stream)
        self.select(key_idx, key_cnt, stream=stream, want_s=want_s)
        return self.compact(hidden, k, v, stream=stream)

    def filter(self, q_text, k, v, hidden, key_idx=None, key_cnt=None, stream=None, want_s=False):
        """The whole step through the single entry point (one launch where the plan allows it)."""
        self._check(mustdrop_filter(self.plan, q_text, k, v, hidden, key_idx, key_cnt, self.g, self.i,
                                    self.s if want_s else None, self.kept_idx, self.kept_cnt,
                                    self.hidden_out if hidden is not None else None, self.k_out,
                                    self.v_out if v is not None else None, self.workspace, stream),
                    "mustdrop_filter")
        return self.hidden_out, self.k_out, self.v_out

    def filter_layer(self, q_text, k, v, hidden, key_idx=None, key_cnt=None, vis_cnt=None, orig_idx=None,
                     stream=None, want_s=False):
        """One layer of a chain (ragged token counts, original ids, key positions for the next layer)."""
        self._check(mustdrop_filter_layer(
            self.plan, self.workspace, stream, q_text=q_text, k=k, v=v, hidden=hidden, key_idx=key_idx,
            key_cnt=key_cnt, vis_cnt=vis_cnt, orig_idx=orig_idx, g_out=self.g, i_out=self.i,
            s_out=self.s if want_s else None, kept_idx=self.kept_idx, kept_cnt=self.kept_cnt, orig_out=self.orig_out,
            key_idx_out=self.key_idx_out if self.config.key_max > 0 else None,
            key_cnt_out=self.key_cnt_out if self.config.key_max > 0 else None,
            hidden_out=self.hidden_out if hidden is not None else None, k_out=self.k_out,
            v_out=self.v_out if v is not None else None), "mustdrop_filter_layer")
        return self.hidden_out, self.k_out, self.v_out

    @property
    def filter_launches(self) -> int:
        return mustdrop_plan_filter_launches(self.plan)

    def device_status(self, stream=None):
        st, code, detail = mustdrop_device_status(self.plan, self.workspace, stream)
        self._check(st, "mustdrop_device_status")
        return code, detail

    @property
    def description(self) -> str:
        return mustdrop_plan_describe(self.plan)

    @property
    def score_variant(self) -> str:
        return mustdrop_plan_score_variant(self.plan)


def config_for(w, **overrides) -> Config:
    """Config of a synth.Workload (sizes only)."""
    base = dict(batch=w.batch, n_heads=w.n_heads, hidden=w.hidden, seq_len=w.seq_len, vis_start=w.vis_start,
                n_vis=w.n_vis, txt_start=w.txt_start, n_txt=w.n_txt, head_dim=w.head_dim, budget=w.budget,
                key_max=max(w.key_cnt, 0))
    base.update(overrides)
    return Config(**base)
