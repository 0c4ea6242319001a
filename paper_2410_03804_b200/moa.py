"""Thin ctypes binding over libmoa.so (the C ABI declared in include/moa.h).

Argument marshalling only: torch provides device memory and streams, every step
of the drafter forward runs in the library's CUDA kernels. There is no CPU or
PyTorch fallback: if the library is missing or no sm_100 GPU is present, the
calls fail loudly.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

MOA_MAX_BATCH = 64
STATUS_NAMES = ["OK", "ERR_NULL", "ERR_SHAPE", "ERR_DTYPE", "ERR_ALIGN", "ERR_WORKSPACE", "ERR_CAPACITY",
                "ERR_STATE", "ERR_ARCH", "ERR_CUDA", "ERR_TIMEOUT"]
MOA_OK = 0

EXPORTS = ["moa_create", "moa_destroy", "moa_tli_configure", "moa_state_bytes", "moa_status_str", "moa_last_cuda_error",
           "moa_state_set_len", "moa_lsa_forward", "moa_sa_append", "moa_sa_append_static", "moa_drafter_prefill", "moa_tree_begin", "moa_draft_step",
           "moa_tree_expand", "moa_tree_attn_mask", "moa_verify_greedy", "moa_pack_tree", "moa_unpack_tree", "moa_quantize_rows", "moa_dequantize_rows", "moa_state_status", "moa_profile_begin", "moa_profile_end", "moa_profile_phases",
           "moa_launch_count", "moa_trace_begin", "moa_trace_end"]


class MoaConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "d_model", "n_stack", "d_stack", "vocab", "head_dim", "lsa_hq", "lsa_hkv", "lsa_mlp",
        "sa_hq", "sa_hkv", "sa_mlp", "ca_hq", "ca_hkv", "ca_mlp", "max_batch", "max_ctx",
        "tree_topk", "tree_depth", "tree_keep")] + [("rms_eps", C.c_float), ("sa_rope_theta", C.c_float),
                                                    ("dtype", C.c_int32)]


WEIGHT_FIELDS = ["embed", "lm_head", "final_norm",
                 "lsa_norm1", "lsa_wq", "lsa_wk", "lsa_wv", "lsa_wo", "lsa_norm2", "lsa_wgate", "lsa_wup", "lsa_wdown",
                 "sa_norm1", "sa_wq", "sa_wk", "sa_wv", "sa_wo", "sa_norm2", "sa_wgate", "sa_wup", "sa_wdown",
                 "ca_normq", "ca_normkv", "ca_wq", "ca_wk", "ca_wv", "ca_wo", "ca_norm2", "ca_wgate", "ca_wup",
                 "ca_wdown"]


class MoaWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_FIELDS]


MOA_MAX_TLI = 4
TLI_LAYER_FIELDS = ["norm1", "wq", "wk", "wv", "wo", "norm2", "wgate", "wup", "wdown"]


class MoaTliConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("hq", C.c_int32), ("hkv", C.c_int32), ("mlp", C.c_int32),
                ("rope_theta", C.c_float)]


class MoaTliLayer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in TLI_LAYER_FIELDS]


class MoaTliCaches(C.Structure):
    _fields_ = [("k", C.c_void_p * MOA_MAX_TLI), ("v", C.c_void_p * MOA_MAX_TLI)]


class MoaState(C.Structure):
    _fields_ = [("ca_k", C.c_void_p), ("ca_v", C.c_void_p), ("sa_k", C.c_void_p), ("sa_v", C.c_void_p),
                ("ca_len", C.c_void_p), ("sa_len", C.c_void_p), ("tree", C.c_void_p),
                ("ca_len_host", C.c_void_p), ("sa_len_host", C.c_void_p), ("step", C.c_int32)]


class MoaError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{what}: MOA_{name}" + (f" ({detail})" if detail else ""))


_lib = None


def lib_path() -> str:
    return _build.LIB


def load_library(rebuild_if_stale: bool = True) -> C.CDLL:
    """Loads libmoa.so, building it first if it is missing or older than its sources and nvcc is around."""
    global _lib
    if _lib is not None:
        return _lib
    trace = os.environ.get("MOA_TRACE_BUILD", "") == "1"          # the variant whose kernels stamp the stage trace
    checks = os.environ.get("MOA_CHECKS_BUILD", "") == "1"        # the debug variant with device-side index checks
    path = _build.LIB_TRACE if trace else _build.LIB_CHECKS if checks else _build.LIB
    if rebuild_if_stale and (os.path.exists("/usr/local/cuda/bin/nvcc") or os.environ.get("NVCC")):
        path = _build.build(trace=trace, checks=checks)
    if not os.path.exists(path):
        raise RuntimeError(f"{path} not found: build it with `python -m paper_2410_03804_b200.build`")
    lib = C.CDLL(path)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    lib.moa_create.argtypes = [C.POINTER(MoaConfig), C.POINTER(MoaWeights), C.POINTER(vp)]
    lib.moa_destroy.argtypes = [vp]
    lib.moa_destroy.restype = None
    lib.moa_state_bytes.argtypes = [vp, i32, C.POINTER(sz), C.POINTER(sz)]
    lib.moa_status_str.argtypes = [i32]
    lib.moa_status_str.restype = C.c_char_p
    lib.moa_last_cuda_error.argtypes = []
    lib.moa_last_cuda_error.restype = C.c_char_p
    lib.moa_tli_configure.argtypes = [vp, C.POINTER(MoaTliConfig), vp, C.POINTER(MoaTliCaches)]
    lib.moa_state_set_len.argtypes = [vp, C.POINTER(MoaState), i32, vp, i32, vp]
    lib.moa_lsa_forward.argtypes = [vp, C.POINTER(MoaState), vp, vp, i32, vp, vp, sz, vp]
    lib.moa_sa_append.argtypes = [vp, C.POINTER(MoaState), vp, vp, i32, vp, sz, vp]
    lib.moa_drafter_prefill.argtypes = [vp, C.POINTER(MoaState), vp, vp, i32, vp, vp, vp, sz, vp]
    lib.moa_sa_append_static.argtypes = [vp, C.POINTER(MoaState), vp, vp, i32, vp]
    lib.moa_tree_begin.argtypes = [vp, C.POINTER(MoaState), vp, i32, vp]
    lib.moa_draft_step.argtypes = [vp, C.POINTER(MoaState), i32, vp, vp, vp, vp, sz, vp]
    lib.moa_tree_expand.argtypes = [vp, C.POINTER(MoaState), i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.moa_tree_attn_mask.argtypes = [vp, i32, i32, vp, i32, vp]
    lib.moa_verify_greedy.argtypes = [vp, vp, i32, i32, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.moa_pack_tree.argtypes = [vp, vp, C.c_int64, vp, vp]
    lib.moa_unpack_tree.argtypes = [vp, C.c_int64, vp, vp, vp]
    lib.moa_quantize_rows.argtypes = [vp, i32, C.c_int64, i32, vp, vp, vp]
    lib.moa_dequantize_rows.argtypes = [vp, vp, C.c_int64, i32, vp, i32, vp]
    lib.moa_state_status.argtypes = [vp, C.POINTER(MoaState), vp]
    lib.moa_profile_begin.argtypes = [vp]
    lib.moa_profile_end.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i32)]
    lib.moa_profile_phases.argtypes = [vp, vp, sz, i32, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(i32),
                                       C.POINTER(i32), vp]
    lib.moa_launch_count.argtypes = []
    lib.moa_trace_begin.argtypes = [vp, i32]
    lib.moa_trace_end.argtypes = [C.POINTER(i32)]
    for n in EXPORTS:
        if n not in ("moa_destroy", "moa_status_str", "moa_last_cuda_error", "moa_launch_count"):
            getattr(lib, n).restype = i32
    lib.moa_launch_count.restype = C.c_int64
    _lib = lib
    return lib


def _check(status: int, what: str):
    if status != MOA_OK:
        detail = load_library().moa_last_cuda_error().decode() if status in (5, 9) else ""
        raise MoaError(status, what, detail)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _host_i32(vals):
    arr = (C.c_int32 * len(vals))(*[int(v) for v in vals])
    return arr


def moa_tree_attn_mask(parent: torch.Tensor, packed: bool = False, stream=None) -> torch.Tensor:
    """Ancestor-or-self mask of a batch of trees. parent: int32 cuda [batch, n]."""
    assert parent.is_cuda and parent.dtype == torch.int32 and parent.dim() == 2 and parent.is_contiguous()
    batch, n = parent.shape
    if packed:
        out = torch.empty((batch, n, (n + 63) // 64), dtype=torch.int64, device=parent.device)
    else:
        out = torch.empty((batch, n, n), dtype=torch.uint8, device=parent.device)
    st = load_library().moa_tree_attn_mask(_ptr(parent), batch, n, _ptr(out) if out.numel() else C.c_void_p(16),
                                           1 if packed else 0, _stream(stream))
    _check(st, "moa_tree_attn_mask")
    return out


def moa_verify_greedy(tok: torch.Tensor, parent: torch.Tensor, target_logits: torch.Tensor, cap: int, out=None,
                      stream=None):
    """tok, parent: cuda int32 [batch, n] (the kept tree); target_logits: cuda float32 / bfloat16 [batch, n, V].
    Returns (choice [batch, n], acc_slot [batch, cap], acc_tok [batch, cap], acc_len [batch], next_tok [batch]);
    out: the same five int32 tensors preallocated by the caller."""
    assert tok.is_cuda and tok.dtype == torch.int32 and tok.is_contiguous() and tok.dim() == 2
    assert parent.is_cuda and parent.dtype == torch.int32 and parent.is_contiguous() and parent.shape == tok.shape
    assert target_logits.is_cuda and target_logits.is_contiguous() and target_logits.shape[:2] == tok.shape
    assert target_logits.dtype in (torch.float32, torch.bfloat16)
    b, n = tok.shape
    dev = tok.device
    if out is not None:
        choice, acc_slot, acc_tok, acc_len, next_tok = out
    else:
        choice = torch.empty((b, n), dtype=torch.int32, device=dev)
        acc_slot = torch.empty((b, cap), dtype=torch.int32, device=dev)
        acc_tok = torch.empty((b, cap), dtype=torch.int32, device=dev)
        acc_len = torch.empty((b,), dtype=torch.int32, device=dev)
        next_tok = torch.empty((b,), dtype=torch.int32, device=dev)
    _check(load_library().moa_verify_greedy(_ptr(tok), _ptr(parent), b, n, _ptr(target_logits),
                                            0 if target_logits.dtype == torch.float32 else 1, target_logits.shape[2],
                                            int(cap), _ptr(choice), _ptr(acc_slot), _ptr(acc_tok), _ptr(acc_len),
                                            _ptr(next_tok), _stream(stream)), "moa_verify_greedy")
    return choice, acc_slot, acc_tok, acc_len, next_tok


def moa_pack_tree(tok: torch.Tensor, parent: torch.Tensor, stream=None) -> torch.Tensor:
    """cuda int32 [..., n] token ids and parent slots -> cuda uint8 [..., n, 4] (the client's 4-bytes-per-node message)."""
    assert tok.is_cuda and tok.dtype == torch.int32 and tok.is_contiguous() and parent.shape == tok.shape
    assert parent.is_cuda and parent.dtype == torch.int32 and parent.is_contiguous()
    msg = torch.empty(tuple(tok.shape) + (4,), dtype=torch.uint8, device=tok.device)
    _check(load_library().moa_pack_tree(_ptr(tok), _ptr(parent), tok.numel(), _ptr(msg), _stream(stream)), "moa_pack_tree")
    return msg


def moa_unpack_tree(msg: torch.Tensor, stream=None):
    assert msg.is_cuda and msg.dtype == torch.uint8 and msg.is_contiguous() and msg.shape[-1] == 4
    tok = torch.empty(tuple(msg.shape[:-1]), dtype=torch.int32, device=msg.device)
    parent = torch.empty_like(tok)
    _check(load_library().moa_unpack_tree(_ptr(msg), tok.numel(), _ptr(tok), _ptr(parent), _stream(stream)), "moa_unpack_tree")
    return tok, parent


def moa_quantize_rows(x: torch.Tensor, out=None, stream=None):
    """x cuda float32 / bfloat16 [rows, width] -> (int8 codes [rows, width], float32 scales [rows])."""
    assert x.is_cuda and x.is_contiguous() and x.dim() == 2 and x.dtype in (torch.float32, torch.bfloat16)
    codes, scales = out if out is not None else (torch.empty(x.shape, dtype=torch.int8, device=x.device),
                                                 torch.empty((x.shape[0],), dtype=torch.float32, device=x.device))
    _check(load_library().moa_quantize_rows(_ptr(x), 0 if x.dtype == torch.float32 else 1, x.shape[0], x.shape[1],
                                            _ptr(codes), _ptr(scales), _stream(stream)), "moa_quantize_rows")
    return codes, scales


def moa_dequantize_rows(codes: torch.Tensor, scales: torch.Tensor, dtype=torch.float32, out=None, stream=None):
    assert codes.is_cuda and codes.dtype == torch.int8 and codes.is_contiguous() and codes.dim() == 2
    assert scales.is_cuda and scales.dtype == torch.float32 and scales.numel() == codes.shape[0]
    if out is None:
        out = torch.empty(codes.shape, dtype=dtype, device=codes.device)
    _check(load_library().moa_dequantize_rows(_ptr(codes), _ptr(scales), codes.shape[0], codes.shape[1], _ptr(out),
                                              0 if out.dtype == torch.float32 else 1, _stream(stream)), "moa_dequantize_rows")
    return out


class MoA:
    """A drafter context plus one decoding state on the current CUDA device.

    weights: dict name -> CUDA tensor (dtype float32 or bfloat16, as cfg['dtype'] says).
    cfg keys: the fields of moa_config except dtype/max_* (given separately). Target Layer Inference: with
    cfg['n_tli'] = N > 0 (plus 'tli_hq', 'tli_hkv', 'tli_mlp') the weights also hold 'tli{l}_{norm1,wq,...}' for
    l < N, and the LLM's caches of those layers are the tensors tli_k[l], tli_v[l] (fill_tli_cache)."""

    def __init__(self, cfg: dict, weights: dict, max_batch: int, max_ctx: int, lsa_chunk_tokens: int = 8):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2410_03804_b200 needs a CUDA device (B200, sm_100a); there is no CPU path")
        self.dtype = torch.float32 if cfg["dtype"] == "f32" else torch.bfloat16
        c = MoaConfig()
        for n in ("d_model", "n_stack", "d_stack", "vocab", "head_dim", "lsa_hq", "lsa_hkv", "lsa_mlp", "sa_hq",
                  "sa_hkv", "sa_mlp", "ca_hq", "ca_hkv", "ca_mlp", "tree_topk", "tree_depth", "tree_keep"):
            setattr(c, n, int(cfg[n]))
        c.max_batch, c.max_ctx = int(max_batch), int(max_ctx)
        c.rms_eps = float(cfg.get("rms_eps", 1e-5))
        c.sa_rope_theta = float(cfg.get("rope_theta", 500000.0))
        c.dtype = 0 if cfg["dtype"] == "f32" else 1
        self.cfg = c
        self.weights = {}
        w = MoaWeights()
        for n in WEIGHT_FIELDS:
            t = weights[n]
            assert t.is_cuda and t.dtype == self.dtype and t.is_contiguous(), n
            self.weights[n] = t          # keep alive
            setattr(w, n, t.data_ptr())
        self._w = w
        h = C.c_void_p()
        _check(self.lib.moa_create(C.byref(c), C.byref(w), C.byref(h)), "moa_create")
        self.h = h
        self.device = weights["embed"].device
        self.n_tli = int(cfg.get("n_tli", 0))
        self.tli_k, self.tli_v = [], []
        if self.n_tli > 0:
            self.moa_tli_configure(cfg, weights, max_batch, max_ctx)
        tb, wb = C.c_size_t(), C.c_size_t()
        _check(self.lib.moa_state_bytes(self.h, int(lsa_chunk_tokens), C.byref(tb), C.byref(wb)), "moa_state_bytes")
        self.tree_bytes, self.ws_bytes = tb.value, wb.value
        dev, dh = self.device, c.head_dim
        self.ca_k = torch.zeros((max_batch, max_ctx, c.ca_hkv, dh), dtype=self.dtype, device=dev)
        self.ca_v = torch.zeros_like(self.ca_k)
        self.sa_k = torch.zeros((max_batch, max_ctx, c.sa_hkv, dh), dtype=self.dtype, device=dev)
        self.sa_v = torch.zeros_like(self.sa_k)
        self.ca_len = torch.zeros(MOA_MAX_BATCH, dtype=torch.int32, device=dev)
        self.sa_len = torch.zeros(MOA_MAX_BATCH, dtype=torch.int32, device=dev)
        self.tree = torch.zeros(self.tree_bytes, dtype=torch.uint8, device=dev)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        self._ca_len_host = (C.c_int32 * MOA_MAX_BATCH)()
        self._sa_len_host = (C.c_int32 * MOA_MAX_BATCH)()
        st = MoaState()
        st.ca_k, st.ca_v, st.sa_k, st.sa_v = (t.data_ptr() for t in (self.ca_k, self.ca_v, self.sa_k, self.sa_v))
        st.ca_len, st.sa_len, st.tree = self.ca_len.data_ptr(), self.sa_len.data_ptr(), self.tree.data_ptr()
        st.ca_len_host = C.addressof(self._ca_len_host)
        st.sa_len_host = C.addressof(self._sa_len_host)
        st.step = -1
        self.st = st

    def close(self):
        if getattr(self, "h", None):
            self.lib.moa_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the C-ABI calls, same names -------------------------------------------------------
    def moa_tli_configure(self, cfg: dict, weights: dict, max_batch: int, max_ctx: int):
        """Turns Target Layer Inference on: binds the N decoder layers' weights and allocates their caches."""
        n = int(cfg["n_tli"])
        tc = MoaTliConfig(n, int(cfg["tli_hq"]), int(cfg["tli_hkv"]), int(cfg["tli_mlp"]),
                          float(cfg.get("rope_theta", 500000.0)))
        layers = (MoaTliLayer * n)()
        for l in range(n):
            for f in TLI_LAYER_FIELDS:
                t = weights[f"tli{l}_{f}"]
                assert t.is_cuda and t.dtype == self.dtype and t.is_contiguous(), (l, f)
                self.weights[f"tli{l}_{f}"] = t
                setattr(layers[l], f, t.data_ptr())
        caches = MoaTliCaches()
        shape = (max_batch, max_ctx, tc.hkv, self.cfg.head_dim)
        self.tli_k = [torch.zeros(shape, dtype=self.dtype, device=self.device) for _ in range(n)]
        self.tli_v = [torch.zeros(shape, dtype=self.dtype, device=self.device) for _ in range(n)]
        for l in range(n):
            caches.k[l], caches.v[l] = self.tli_k[l].data_ptr(), self.tli_v[l].data_ptr()
        _check(self.lib.moa_tli_configure(self.h, C.byref(tc), C.cast(layers, C.c_void_p), C.byref(caches)),
               "moa_tli_configure")

    def moa_state_set_len(self, which: str, lens, stream=None):
        lens = [int(v) for v in lens]
        _check(self.lib.moa_state_set_len(self.h, C.byref(self.st), 0 if which == "ca" else 1, _host_i32(lens),
                                          len(lens), _stream(stream)), "moa_state_set_len")

    def moa_lsa_forward(self, h_stack: torch.Tensor, n_tok, want_kv: bool = True, stream=None):
        """h_stack: T cuda [sum n_tok, S, D_in]; n_tok: list of per-sequence token counts."""
        assert h_stack.is_cuda and h_stack.dtype == self.dtype and h_stack.is_contiguous()
        n_tok = [int(v) for v in n_tok]
        assert h_stack.shape[0] == sum(n_tok)
        kv = torch.empty((sum(n_tok), self.cfg.d_stack), dtype=self.dtype, device=self.device) if want_kv else None
        _check(self.lib.moa_lsa_forward(self.h, C.byref(self.st), _ptr(h_stack), _host_i32(n_tok), len(n_tok),
                                        _ptr(kv), _ptr(self.ws), self.ws_bytes, _stream(stream)), "moa_lsa_forward")
        return kv

    def moa_sa_append(self, tok: torch.Tensor, n, stream=None):
        assert tok.is_cuda and tok.dtype == torch.int32 and tok.is_contiguous()
        n = [int(v) for v in n]
        assert tok.numel() == sum(n)
        _check(self.lib.moa_sa_append(self.h, C.byref(self.st), _ptr(tok), _host_i32(n), len(n), _ptr(self.ws),
                                      self.ws_bytes, _stream(stream)), "moa_sa_append")

    def moa_drafter_prefill(self, tok: torch.Tensor, n, ca_limit=None, out=None, stream=None):
        """The drafter over whole sequences in one pass: tok cuda int32 [sum n]; ca_limit cuda int32 [sum n] or
        None. Returns hidden [sum n, E] and appends the tokens to the self-attention prefix."""
        assert tok.is_cuda and tok.dtype == torch.int32 and tok.is_contiguous()
        n = [int(v) for v in n]
        assert tok.numel() == sum(n)
        if ca_limit is not None:
            assert ca_limit.is_cuda and ca_limit.dtype == torch.int32 and ca_limit.numel() == sum(n)
        hid = out if out is not None else torch.empty((sum(n), self.cfg.d_model), dtype=self.dtype, device=self.device)
        _check(self.lib.moa_drafter_prefill(self.h, C.byref(self.st), _ptr(tok), _host_i32(n), len(n), _ptr(ca_limit),
                                            _ptr(hid), _ptr(self.ws), self.ws_bytes, _stream(stream)), "moa_drafter_prefill")
        return hid

    def moa_sa_append_static(self, tok: torch.Tensor, n, stream=None):
        """moa_sa_append without a workspace: the library's fixed scratch array is used, nothing is allocated.
        For callers that cannot allocate device memory; at most 32 tokens per call (see include/moa.h)."""
        assert tok.is_cuda and tok.dtype == torch.int32 and tok.is_contiguous()
        n = [int(v) for v in n]
        assert tok.numel() == sum(n)
        _check(self.lib.moa_sa_append_static(self.h, C.byref(self.st), _ptr(tok), _host_i32(n), len(n),
                                             _stream(stream)), "moa_sa_append_static")

    def moa_tree_begin(self, root_tok: torch.Tensor, stream=None):
        assert root_tok.is_cuda and root_tok.dtype == torch.int32 and root_tok.is_contiguous()
        self.batch = root_tok.numel()
        _check(self.lib.moa_tree_begin(self.h, C.byref(self.st), _ptr(root_tok), self.batch, _stream(stream)),
               "moa_tree_begin")

    def rows(self) -> int:
        return self.batch if self.st.step == 0 else self.batch * self.cfg.tree_topk

    def moa_draft_step(self, want_hidden: bool = False, out=None, stream=None):
        """Returns (topk_id [R,B] int32, topk_logp [R,B] float32, hidden [R,E] or None)."""
        R, B = self.rows(), self.cfg.tree_topk
        if out is None:
            ids = torch.empty((R, B), dtype=torch.int32, device=self.device)
            lp = torch.empty((R, B), dtype=torch.float32, device=self.device)
            hid = torch.empty((R, self.cfg.d_model), dtype=self.dtype, device=self.device) if want_hidden else None
        else:
            ids, lp, hid = out
        _check(self.lib.moa_draft_step(self.h, C.byref(self.st), self.batch, _ptr(ids), _ptr(lp), _ptr(hid),
                                       _ptr(self.ws), self.ws_bytes, _stream(stream)), "moa_draft_step")
        return ids, lp, hid

    def moa_tree_expand(self, ids: torch.Tensor, lp: torch.Tensor, out=None, stream=None):
        """Expands with the given top-B lists. After the last step returns the kept tree as
        (tok, parent, depth, score, n) tensors of shape [batch, m+1] / [batch]; otherwise None."""
        assert ids.is_cuda and ids.dtype == torch.int32 and lp.dtype == torch.float32
        last = self.st.step + 1 == self.cfg.tree_depth
        outs = out
        if last and outs is None:
            W = self.cfg.tree_keep + 1
            outs = (torch.empty((self.batch, W), dtype=torch.int32, device=self.device),
                    torch.empty((self.batch, W), dtype=torch.int32, device=self.device),
                    torch.empty((self.batch, W), dtype=torch.int32, device=self.device),
                    torch.empty((self.batch, W), dtype=torch.float32, device=self.device),
                    torch.empty((self.batch,), dtype=torch.int32, device=self.device))
        p = [_ptr(t) for t in outs] if outs is not None else [None] * 5
        _check(self.lib.moa_tree_expand(self.h, C.byref(self.st), self.batch, _ptr(ids), _ptr(lp), *p, _stream(stream)),
               "moa_tree_expand")
        return outs if last else None

    def moa_state_status(self, stream=None) -> int:
        return int(self.lib.moa_state_status(self.h, C.byref(self.st), _stream(stream)))

    def moa_profile_begin(self):
        _check(self.lib.moa_profile_begin(self.h), "moa_profile_begin")

    def moa_profile_end(self):
        """Returns (summed LM-head kernel milliseconds, launches timed)."""
        ms, n = C.c_double(), C.c_int32()
        _check(self.lib.moa_profile_end(self.h, C.byref(ms), C.byref(n)), "moa_profile_end")
        return ms.value, n.value

    PHASE_KINDS = ["gemm", "rows_norm", "res_norm", "mean_norm", "cache_append", "lsa_attention"]

    def moa_profile_phases(self, stream=None):
        """[(kind name, microseconds, of which in the closing barrier)] of the last dense LSA pass launched while
        profiling was on."""
        cap = 32
        us, wait, kinds, n = (C.c_double * cap)(), (C.c_double * cap)(), (C.c_int32 * cap)(), C.c_int32()
        _check(self.lib.moa_profile_phases(self.h, _ptr(self.ws), self.ws_bytes, cap, us, wait, kinds, C.byref(n),
                                           _stream(stream)), "moa_profile_phases")
        return [(self.PHASE_KINDS[kinds[i]], us[i], wait[i]) for i in range(n.value)]

    def moa_launch_count(self) -> int:
        return int(self.lib.moa_launch_count())

    TRACE_KINDS = ["other", "embed", "gemm", "attention", "attn_merge", "lm_merge", "tree_expand", "row_norm", "res_norm",
                   "swiglu", "sum_cast", "rope", "cache_append", "layer_mean"]

    def moa_trace_begin(self, cap: int = 4096):
        """Starts the stage trace (library built with MOA_TRACE_BUILD=1 only)."""
        self._trace = torch.zeros(2 * cap, dtype=torch.int64, device=self.device)
        _check(self.lib.moa_trace_begin(_ptr(self._trace), cap), "moa_trace_begin")

    def moa_trace_end(self):
        """[(kernel kind, gridDim.x, nanosecond stamp)] in launch order."""
        n = C.c_int32()
        _check(self.lib.moa_trace_end(C.byref(n)), "moa_trace_end")
        t = self._trace.cpu().tolist()
        return [(self.TRACE_KINDS[(t[2 * i + 1] >> 32) & 0xff], t[2 * i + 1] & 0xffffffff, t[2 * i]) for i in range(min(n.value, len(t) // 2))]

    # ---- convenience for tests / bench: raw views of the tree blob ---------------------------
    def fill_cache(self, which: str, k: torch.Tensor, v: torch.Tensor):
        """Copies caller-made cache content [batch, n, hkv, dh] in and sets the lengths."""
        ck, cv = (self.ca_k, self.ca_v) if which == "ca" else (self.sa_k, self.sa_v)
        b, n = k.shape[0], k.shape[1]
        ck[:b, :n].copy_(k)
        cv[:b, :n].copy_(v)
        self.moa_state_set_len(which, [n] * b)

    def fill_tli_cache(self, layer: int, k: torch.Tensor, v: torch.Tensor):
        """Copies the LLM's cache of one Target-Layer-Inference layer [batch, n, hkv, dh] in (positions 0..n-1;
        the valid length is the self-attention prefix length)."""
        b, n = k.shape[0], k.shape[1]
        self.tli_k[layer][:b, :n].copy_(k)
        self.tli_v[layer][:b, :n].copy_(v)
