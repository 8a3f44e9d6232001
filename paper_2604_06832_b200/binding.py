"""ctypes binding of `libfdvlm.so`: argument marshalling only.

Every function of `include/fdvlm.h` is reachable as `lib().<name>`; the `Handle` class wraps one
`fdvlm_t*` with methods of the same names (without the `fdvlm_` prefix).  PyTorch is used for
device memory and streams.  There is no fallback of any kind: if the shared library is missing or
fails to load, importing callers get an exception.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import inputs as _in

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfdvlm.so")

FDVLM_OK = 0
ERR_INVALID_ARG, ERR_STATE, ERR_CAPACITY, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT, ERR_OOM = -1, -2, -3, -4, -5, -6, -7
DT_F32, DT_BF16, DT_FP8, DT_W8A8 = 0, 1, 2, 3
KV_BF16, KV_F16 = 0, 1
RULE_THRESHOLD, RULE_TOPK = 0, 1
KERNEL_KINDS = ("rope_table", "gemm_qkv", "fin_qkv", "attention", "attn_merge", "gemm_o", "fin_resid", "gemm_gate_up",
                "gemm_down", "gemm_lm_head", "stats_merge")
_DTYPE_CODE = {_in.F32: DT_F32, _in.BF16: DT_BF16, _in.FP8: DT_FP8, _in.W8A8: DT_W8A8}


class Config(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "intermediate",
                                       "vocab", "mask_id")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("tie_embeddings", C.c_int), ("dtype", C.c_int),
                ("max_seq", C.c_int), ("max_block", C.c_int), ("kv_dtype", C.c_int)]


_LW_FIELDS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "bq", "bk", "bv",
              "s_q", "s_k", "s_v", "s_o", "s_gate", "s_up", "s_down", "g_attn", "g_mlp")


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _LW_FIELDS]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("s_lm_head", C.c_void_p), ("g_final", C.c_void_p),
                ("layers", C.POINTER(LayerWeights))]


class StepParams(C.Structure):
    _fields_ = [("rule", C.c_int), ("threshold", C.c_float), ("k", C.c_int), ("pred_shift", C.c_int)]


class StepInfo(C.Structure):
    _fields_ = [("n_unmasked", C.c_int), ("n_remaining", C.c_int), ("step_index", C.c_int)]


class KernelRecord(C.Structure):
    _fields_ = [("kind", C.c_int), ("start_us", C.c_double), ("released_us", C.c_double), ("end_us", C.c_double)]


class SpecInfo(C.Structure):
    _fields_ = [("accepted", C.c_int), ("next_token", C.c_int32), ("cache_len", C.c_int)]


class QuadInfo(C.Structure):
    _fields_ = [("accepted", C.c_int), ("cache_len", C.c_int)]


EXPORTS = {
    "fdvlm_create": (C.c_int, [C.POINTER(Config), C.POINTER(Weights), C.c_void_p, C.POINTER(C.c_void_p)]),
    "fdvlm_destroy": (None, [C.c_void_p]),
    "fdvlm_reset": (C.c_int, [C.c_void_p]),
    "fdvlm_synchronize": (C.c_int, [C.c_void_p]),
    "fdvlm_debug_poison": (C.c_int, [C.c_void_p, C.c_int]),
    "fdvlm_decode_block": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.POINTER(StepParams), C.c_void_p, C.POINTER(StepInfo)]),
    "fdvlm_profile_read_chain": (C.c_int, [C.c_void_p, C.POINTER(KernelRecord), C.c_int, C.POINTER(C.c_int)]),
    "fdvlm_op_linear_status": (C.c_int, [C.c_void_p, C.c_void_p]),
    "fdvlm_prefill": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p]),
    "fdvlm_block_begin": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p]),
    "fdvlm_block_begin_host": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p]),
    "fdvlm_block_step": (C.c_int, [C.c_void_p, C.POINTER(StepParams), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_void_p, C.POINTER(StepInfo)]),
    "fdvlm_block_step_host": (C.c_int, [C.c_void_p, C.POINTER(StepParams), C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.POINTER(StepInfo)]),
    "fdvlm_block_set_tokens": (C.c_int, [C.c_void_p, C.c_void_p]),
    "fdvlm_decode_block_topk": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.POINTER(StepInfo)]),
    "fdvlm_commit_decode_block_topk": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.POINTER(StepInfo)]),
    "fdvlm_commit_decode_block": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.POINTER(StepParams), C.c_void_p, C.POINTER(StepInfo)]),
    "fdvlm_commit_begin_step": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.POINTER(StepParams), C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(StepInfo)]),
    "fdvlm_commit_begin_step_host": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.POINTER(StepParams), C.c_void_p, C.c_void_p,
                                               C.c_void_p, C.c_void_p, C.POINTER(StepInfo)]),
    "fdvlm_commit_block": (C.c_int, [C.c_void_p, C.c_void_p]),
    "fdvlm_commit_block_verify": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "fdvlm_truncate": (C.c_int, [C.c_void_p, C.c_int]),
    "fdvlm_util_stream_read": (C.c_int, [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]),
    "fdvlm_spec_block": (C.c_int, [C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(SpecInfo)]),
    "fdvlm_quad_begin": (C.c_int, [C.c_void_p, C.c_int, C.c_int32, C.c_int, C.c_void_p]),
    "fdvlm_quad_set_draft": (C.c_int, [C.c_void_p, C.c_void_p]),
    "fdvlm_quad_step": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(QuadInfo)]),
    "fdvlm_quad_end": (C.c_int, [C.c_void_p]),
    "fdvlm_cache_len": (C.c_int, [C.c_void_p]),
    "fdvlm_cache_read": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p]),
    "fdvlm_last_launch_count": (C.c_int, [C.c_void_p]),
    "fdvlm_last_error": (C.c_char_p, [C.c_void_p]),
    "fdvlm_profile_enable": (C.c_int, [C.c_void_p, C.c_int]),
    "fdvlm_profile_read": (C.c_int, [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int), C.POINTER(C.c_double),
                                     C.POINTER(C.c_int)]),
    "fdvlm_op_linear": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                  C.c_int, C.c_void_p, C.c_void_p]),
    "fdvlm_op_linear_static": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                         C.c_int, C.c_void_p]),
    "fdvlm_op_linear_workspace_bytes": (C.c_size_t, [C.c_int, C.c_int, C.c_int, C.c_int]),
    "fdvlm_op_attention": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int,
                                     C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p]),
    "fdvlm_op_attention_workspace_bytes": (C.c_size_t, [C.c_int, C.c_int, C.c_int, C.c_int]),
    "fdvlm_version": (C.c_char_p, []),
}

_lib = None


def lib() -> C.CDLL:
    """The loaded C-ABI library (loads it on first use; raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2604_06832_b200.build` (no fallback exists)")
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(l, name)
            fn.restype, fn.argtypes = res, args
        _lib = l
    return _lib


class FdvlmError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"fdvlm error {code}: {msg}")
        self.code = code


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> Optional[int]:
    return None if stream is None else stream.cuda_stream


def weights_to_device(weights: dict, device="cuda") -> dict:
    """Copy the CPU weight dict of `inputs.make_weights` to the GPU (same structure)."""
    out = {k: (v.to(device) if isinstance(v, torch.Tensor) else v) for k, v in weights.items() if k != "layers"}
    out["layers"] = [{k: (v.to(device) if isinstance(v, torch.Tensor) else v) for k, v in lw.items()}
                     for lw in weights["layers"]]
    return out


class Handle:
    """One request (batch size one).  `weights` is a dict of CUDA tensors laid out as by
    `inputs.make_weights`; it is kept alive by this object because the library borrows the pointers."""

    def __init__(self, shape: _in.ModelShape, weights: dict, max_seq: int, max_block: int = 64,
                 stream: Optional[torch.cuda.Stream] = None, kv_dtype: int = KV_F16):
        self.shape, self.weights, self.stream = shape, weights, stream
        self.max_seq, self.max_block = max_seq, max_block
        self.kv_dtype = kv_dtype
        cfg = Config(shape.n_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                     shape.intermediate, shape.vocab, shape.mask_id, shape.rms_eps, shape.rope_theta,
                     int(shape.tie_embeddings), _DTYPE_CODE[shape.dtype], max_seq, max_block, kv_dtype)
        self._layers = (LayerWeights * shape.n_layers)()
        for i, lw in enumerate(weights["layers"]):
            for name in _LW_FIELDS:
                setattr(self._layers[i], name, _ptr(lw.get(name)))
        w = Weights(_ptr(weights["embed"]), _ptr(weights.get("lm_head")), _ptr(weights.get("s_lm_head")),
                    _ptr(weights["g_final"]), self._layers)
        self._h = C.c_void_p()
        rc = lib().fdvlm_create(C.byref(cfg), C.byref(w), _stream_ptr(stream), C.byref(self._h))
        if rc != FDVLM_OK:
            raise FdvlmError(rc, lib().fdvlm_last_error(None).decode())
        self.act_dtype = torch.float32 if shape.dtype == _in.F32 else torch.bfloat16
        self.kv_torch_dtype = torch.float32 if shape.dtype == _in.F32 else (torch.float16 if kv_dtype == KV_F16 else torch.bfloat16)

    def _check(self, rc: int):
        if rc != FDVLM_OK:
            raise FdvlmError(rc, lib().fdvlm_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            lib().fdvlm_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        self._check(lib().fdvlm_reset(self._h))

    def synchronize(self):
        self._check(lib().fdvlm_synchronize(self._h))

    def debug_poison(self, on: bool):
        self._check(lib().fdvlm_debug_poison(self._h, int(on)))

    def decode_block(self, block_size: int, rule: int, threshold: float = 0.9, k: int = 8,
                     init_tokens: Optional[torch.Tensor] = None, pred_shift: int = 0,
                     block_tokens: Optional[torch.Tensor] = None) -> StepInfo:
        p, info = StepParams(rule, threshold, k, pred_shift), StepInfo()
        self._check(lib().fdvlm_decode_block(self._h, block_size, _ptr(init_tokens), C.byref(p), _ptr(block_tokens), C.byref(info)))
        return info

    def prefill(self, embeds: Optional[torch.Tensor], tokens: Optional[torch.Tensor],
                last_logits: Optional[torch.Tensor] = None):
        ne = 0 if embeds is None else embeds.shape[0]
        nt = 0 if tokens is None else tokens.shape[0]
        self._check(lib().fdvlm_prefill(self._h, _ptr(embeds), ne, _ptr(tokens), nt, _ptr(last_logits)))

    def block_begin(self, block_size: int, init_tokens: Optional[torch.Tensor] = None):
        self._check(lib().fdvlm_block_begin(self._h, block_size, _ptr(init_tokens)))

    def block_begin_host(self, block_size: int, init_tokens_host: Optional[torch.Tensor] = None):
        self._check(lib().fdvlm_block_begin_host(self._h, block_size, _ptr(init_tokens_host)))

    def block_step(self, rule: int, threshold: float = 0.9, k: int = 8, logits=None, conf=None, pred=None,
                   unmask=None, block_tokens=None, pred_shift: int = 0) -> StepInfo:
        p, info = StepParams(rule, threshold, k, pred_shift), StepInfo()
        self._check(lib().fdvlm_block_step(self._h, C.byref(p), _ptr(logits), _ptr(conf), _ptr(pred), _ptr(unmask),
                                           _ptr(block_tokens), C.byref(info)))
        self._remaining = info.n_remaining
        return info

    def last_info_remaining(self) -> int:
        """n_remaining reported by the last block_step of this wrapper."""
        return getattr(self, "_remaining", 0)

    def block_step_host(self, rule: int, threshold: float = 0.9, k: int = 8, conf=None, pred=None, unmask=None,
                        block_tokens=None, pred_shift: int = 0) -> StepInfo:
        p, info = StepParams(rule, threshold, k, pred_shift), StepInfo()
        self._check(lib().fdvlm_block_step_host(self._h, C.byref(p), _ptr(conf), _ptr(pred), _ptr(unmask),
                                                _ptr(block_tokens), C.byref(info)))
        return info

    def commit_begin_step(self, next_block_size: int, rule: int, threshold: float = 0.9, k: int = 8, next_logits=None,
                          next_init_tokens=None, logits=None, conf=None, pred=None, unmask=None, block_tokens=None,
                          pred_shift: int = 0) -> StepInfo:
        p, info = StepParams(rule, threshold, k, pred_shift), StepInfo()
        self._check(lib().fdvlm_commit_begin_step(self._h, _ptr(next_logits), next_block_size, _ptr(next_init_tokens), C.byref(p),
                                                  _ptr(logits), _ptr(conf), _ptr(pred), _ptr(unmask), _ptr(block_tokens),
                                                  C.byref(info)))
        self._remaining = info.n_remaining
        return info

    def commit_begin_step_host(self, next_block_size: int, rule: int, threshold: float = 0.9, k: int = 8, next_init_tokens=None,
                               conf=None, pred=None, unmask=None, block_tokens=None, pred_shift: int = 0) -> StepInfo:
        p, info = StepParams(rule, threshold, k, pred_shift), StepInfo()
        self._check(lib().fdvlm_commit_begin_step_host(self._h, next_block_size, _ptr(next_init_tokens), C.byref(p), _ptr(conf),
                                                       _ptr(pred), _ptr(unmask), _ptr(block_tokens), C.byref(info)))
        return info

    def commit_decode_block(self, block_size: int, rule: int, threshold: float = 0.9, k: int = 8,
                            init_tokens: Optional[torch.Tensor] = None, pred_shift: int = 0,
                            block_tokens: Optional[torch.Tensor] = None) -> StepInfo:
        p, info = StepParams(rule, threshold, k, pred_shift), StepInfo()
        self._check(lib().fdvlm_commit_decode_block(self._h, block_size, _ptr(init_tokens), C.byref(p), _ptr(block_tokens),
                                                    C.byref(info)))
        return info

    def commit_decode_block_topk(self, block_size: int, k: int, init_tokens: Optional[torch.Tensor] = None, pred_shift: int = 0,
                                 block_tokens: Optional[torch.Tensor] = None) -> StepInfo:
        info = StepInfo()
        self._check(lib().fdvlm_commit_decode_block_topk(self._h, block_size, _ptr(init_tokens), k, pred_shift,
                                                         _ptr(block_tokens), C.byref(info)))
        return info

    def decode_block_topk(self, block_size: int, k: int, init_tokens: Optional[torch.Tensor] = None, pred_shift: int = 0,
                          block_tokens: Optional[torch.Tensor] = None) -> StepInfo:
        info = StepInfo()
        self._check(lib().fdvlm_decode_block_topk(self._h, block_size, _ptr(init_tokens), k, pred_shift, _ptr(block_tokens),
                                                  C.byref(info)))
        return info

    def block_set_tokens(self, tokens: torch.Tensor):
        self._check(lib().fdvlm_block_set_tokens(self._h, _ptr(tokens)))

    def commit_block(self, next_logits: Optional[torch.Tensor] = None):
        self._check(lib().fdvlm_commit_block(self._h, _ptr(next_logits)))

    def commit_block_verify(self, row_pred: Optional[torch.Tensor] = None, row_conf: Optional[torch.Tensor] = None,
                            next_logits: Optional[torch.Tensor] = None):
        self._check(lib().fdvlm_commit_block_verify(self._h, _ptr(row_pred), _ptr(row_conf), _ptr(next_logits)))

    def truncate(self, new_len: int):
        self._check(lib().fdvlm_truncate(self._h, new_len))

    def spec_block(self, block_size: int, seed_token: int, draft_tokens: Optional[torch.Tensor] = None,
                   verify_pred: Optional[torch.Tensor] = None) -> SpecInfo:
        info = SpecInfo()
        self._check(lib().fdvlm_spec_block(self._h, block_size, seed_token, _ptr(draft_tokens), _ptr(verify_pred),
                                           C.byref(info)))
        return info

    def quad_begin(self, block_size: int, first_token: int, chain: bool = False, draft: Optional[torch.Tensor] = None):
        self._check(lib().fdvlm_quad_begin(self._h, block_size, first_token, int(chain), _ptr(draft)))

    def quad_set_draft(self, draft: torch.Tensor):
        self._check(lib().fdvlm_quad_set_draft(self._h, _ptr(draft)))

    def quad_step(self, accepted_tokens: Optional[torch.Tensor] = None, next_draft: Optional[torch.Tensor] = None,
                  row_pred: Optional[torch.Tensor] = None, logits: Optional[torch.Tensor] = None) -> QuadInfo:
        info = QuadInfo()
        self._check(lib().fdvlm_quad_step(self._h, _ptr(accepted_tokens), _ptr(next_draft), _ptr(row_pred), _ptr(logits),
                                          C.byref(info)))
        return info

    def quad_end(self):
        self._check(lib().fdvlm_quad_end(self._h))

    def cache_len(self) -> int:
        return lib().fdvlm_cache_len(self._h)

    def cache_read(self, layer: int, which: int, pos0: int, n: int) -> torch.Tensor:
        dst = torch.empty(n, self.shape.n_kv_heads, self.shape.head_dim, dtype=self.kv_torch_dtype, device="cuda")
        self._check(lib().fdvlm_cache_read(self._h, layer, which, pos0, n, _ptr(dst)))
        return dst

    def last_launch_count(self) -> int:
        return lib().fdvlm_last_launch_count(self._h)

    def profile_enable(self, mode):
        self._check(lib().fdvlm_profile_enable(self._h, int(mode)))

    def profile_read_chain(self, cap: int = 1024) -> list:
        """Records of the last forward under profile mode 2: dicts(kind, start_us, released_us, end_us) in launch order."""
        recs, n = (KernelRecord * cap)(), C.c_int()
        self._check(lib().fdvlm_profile_read_chain(self._h, recs, cap, C.byref(n)))
        return [dict(kind=KERNEL_KINDS[r.kind], start_us=r.start_us, released_us=r.released_us, end_us=r.end_us)
                for r in recs[:min(n.value, cap)]]

    def profile_read(self) -> dict:
        ml, ma, nl, na = C.c_double(), C.c_double(), C.c_int(), C.c_int()
        self._check(lib().fdvlm_profile_read(self._h, C.byref(ml), C.byref(nl), C.byref(ma), C.byref(na)))
        return dict(ms_linear=ml.value, n_linear=nl.value, ms_attention=ma.value, n_attention=na.value)


def util_stream_read(buf: torch.Tensor, sink: torch.Tensor, stream: Optional[torch.cuda.Stream] = None):
    rc = lib().fdvlm_util_stream_read(_ptr(buf), buf.numel() * buf.element_size(), _ptr(sink), _stream_ptr(stream))
    if rc != FDVLM_OK:
        raise FdvlmError(rc, "fdvlm_util_stream_read")


def op_linear(x: torch.Tensor, w: torch.Tensor, scale=None, bias=None, dtype: int = DT_BF16,
              stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    m, k = x.shape
    n = w.shape[0]
    y = torch.empty(m, n, dtype=torch.float32, device=x.device)
    nbytes = lib().fdvlm_op_linear_workspace_bytes(m, n, k, dtype)
    ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=x.device)
    rc = lib().fdvlm_op_linear(_ptr(x), _ptr(w), _ptr(scale), _ptr(bias), _ptr(y), m, n, k, dtype, _ptr(ws),
                               _stream_ptr(stream))
    if rc == FDVLM_OK:
        rc = lib().fdvlm_op_linear_status(_ptr(ws), _stream_ptr(stream))
    if rc != FDVLM_OK:
        raise FdvlmError(rc, "fdvlm_op_linear")
    return y


def op_linear_static(x: torch.Tensor, w: torch.Tensor, scale=None, bias=None, dtype: int = DT_BF16,
                     stream: Optional[torch.cuda.Stream] = None, y: Optional[torch.Tensor] = None) -> torch.Tensor:
    """`fdvlm_op_linear_static`: same result as `op_linear`, scratch taken from the library's built-in device
    array, so the call itself allocates nothing (pass `y` to keep this wrapper from allocating the output)."""
    m, k = x.shape
    n = w.shape[0]
    if y is None:
        y = torch.empty(m, n, dtype=torch.float32, device=x.device)
    rc = lib().fdvlm_op_linear_static(_ptr(x), _ptr(w), _ptr(scale), _ptr(bias), _ptr(y), m, n, k, dtype, _stream_ptr(stream))
    if rc == FDVLM_OK:
        rc = lib().fdvlm_op_linear_status(None, _stream_ptr(stream))
    if rc != FDVLM_OK:
        raise FdvlmError(rc, lib().fdvlm_last_error(None).decode())
    return y


def op_attention(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, cache_len: int, causal: bool,
                 dtype: int = DT_BF16, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Element type of q / caches / result: fp32 with DT_F32, else the tensors' own 16-bit type (bf16 or f16)."""
    kv = KV_F16 if q.dtype == torch.float16 else KV_BF16
    n, hq, d = q.shape
    hkv, max_seq, _ = k_cache.shape
    out = torch.empty(n, hq * d, dtype=q.dtype, device=q.device)
    nbytes = lib().fdvlm_op_attention_workspace_bytes(n, hq, hkv, d)
    ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=q.device)
    rc = lib().fdvlm_op_attention(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(out), n, cache_len, max_seq, hq, hkv, d,
                                  int(causal), dtype, kv, _ptr(ws), _stream_ptr(stream))
    if rc != FDVLM_OK:
        raise FdvlmError(rc, "fdvlm_op_attention")
    return out
